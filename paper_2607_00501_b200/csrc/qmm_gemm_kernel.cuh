// qmm_gemm_kernel.cuh -- tensor-core product of packed Q4/Q8 weights with fp16
// activations, shared by the dense prefill GEMM and the grouped expert GEMMs.
//
// The paper's prefill kernels are tiled GEMMs that dequantise in the inner
// loop (Sec. 3.3, Sec. 3.4).  On B200 the contraction runs on tcgen05 tensor
// cores, which cannot read 4/8-bit codes with fp16 block scales, so CUDA cores
// expand codes to fp16 weights and hand them to the tensor core *through
// tensor memory*: tcgen05.mma takes its A operand from TMEM, so the expanded
// weights never touch shared memory or L2.
//
// Orientation.  Weights sit on the MMA M axis (128 rows = 128 TMEM lanes, one
// weight row per lane -- the same "one row per lane" order the packed layout
// has), tokens on the MMA N axis:  D[n, m] = sum_k W[n, k] * X[m, k].
//
// One thread block computes NA (1 or 2) weight tiles of 128 rows against one
// tile of BN tokens; with NA = 2 both weight tiles reuse the same activation
// tile (half the activation traffic; the gate and up matrices of an expert).
//
// Roles (warp specialised):
//   expanders (8 warps; 16 for token tiles of 64 and narrower and for two tile
//                      sets): several per weight tile and lane
//                      quarter, alternating stages; thread = one weight row;
//                      32-byte code loads straight from global/L2, unpack to
//                      fp16(d*q), tcgen05.st into the A ring in TMEM.
//   epilogue (8 warps, two per lane quarter; 4 where there are 16 expanders):
//                      tcgen05.ld the accumulators, convert, stage the tile in
//                      shared memory as fp16, release the accumulators, then
//                      store the tile with 16-byte row segments (or SiLU*mul of
//                      the staged gate and up values).
//   TMA producer (1 warp): activation tiles -> shared-memory ring (128-byte
//                      swizzle), one lane.
//   MMA issuer (1 warp per weight tile set, converged): tcgen05.mma
//                      (M128 x N x K16, N = the piece's
//                      valid token rows rounded up to 16) and the
//                      tcgen05.commit that frees a ring slot, predicated on one
//                      elected lane (no divergent branch around them).
// The kernel is persistent: a block loops over tiles and the pipeline runs on
// across tile boundaries.
//
// TMEM columns: one or two accumulator buffers of NA*BN fp32 columns, then
// STAGES slots of NA*32 columns (64 fp16 k-values per row and weight tile).
// Activation tiles share those stages (one `full` and one `empty` barrier per
// stage for both operands) except where tensor memory leaves only 3-4 weight
// slots: there they have a deeper ring and barriers of their own (kSplit).
//
// Every mbarrier wait is bounded; on give-up the block raises an abort flag,
// records QMM_ERR_DEVICE_TIMEOUT in the status word, stops issuing work, waits
// (bounded) for its outstanding TMA loads, frees its TMEM and returns.
#pragma once

#include "qmm_common.cuh"
#include "qmm_tc.cuh"

namespace qmm {

constexpr int kGemmBK = 64;          // k per pipeline stage
constexpr int kGemmMaxStagesB = 8;    // depth of the activation ring where it is a ring of its own
constexpr int kGemmMaxStages = 6;     // pipeline depth is min(this, what tensor memory leaves for the weight ring)

#ifndef QMM_GEMM_PREFETCH
#define QMM_GEMM_PREFETCH 2
#endif
constexpr int kGemmPrefetch = QMM_GEMM_PREFETCH;   // weight slices in flight per expander thread (default)

enum GemmEpilogue { kEpiStore = 0, kEpiSiluMul = 1 };

struct GemmParams {
    const uint8_t* w[2];             // packed weights of tile set 0 / 1 (expert 0)
    int64_t w_expert_stride;         // bytes between experts (grouped), else 0
    int N, K;                        // weight matrix [N, K] (per expert)
    uint16_t* out;                   // [rows, ldo] fp16
    int64_t ldo;
    int a_col_offset;                // output column offset of tile set 1 (plain store epilogue)
    int M;                           // rows of X / out (dense); capacity of the row space (grouped)
    // grouped mode (tile_expert != nullptr): token tiles come from a device-built list
    const int* tile_expert;          // [max_tiles] expert of token tile y
    const int* tile_row0;            // [max_tiles] first permuted row of the tile
    const int* tile_rows;            // [max_tiles] valid rows in the tile (<= BN)
    const int* num_tiles;            // [1]
    // dense mode: block b takes whole_tiles / grid whole tiles, then the units [b*U, (b+1)*U) of the
    // tile-major sequence of (tile, k-block) units of the remaining tiles; the pieces of a tile cut
    // by a block boundary go to `partial` as fp32 and a second kernel adds them
    int whole_tiles;                 // the first whole_tiles tiles (a multiple of the grid size) are dealt whole, contiguously
    int tail_halves;                 // != 0: the remaining tiles are dealt as halves of BN / 2 tokens, one after the other over the blocks
    int units_per_block;             // U: share of the (tile, k-block) units of the other tiles
    float* partial;                  // [2 * gridDim.x] slots of NA*BN*128 floats (when some tile is cut)
    // Grouped products of one layer handed over tile by tile instead of kernel by kernel.  sync[0] is set
    // once the token-tile list may be read; sync[1 + mt] counts the epilogue warps of the producing
    // product (gate/up) that have stored their part of token tile mt.  The consuming product (down)
    // starts under programmatic dependent launch on the SMs the producer's last round leaves idle, reads
    // the list once sync[0] is set and loads token tile mt once its counter has reached sync_need.
    int* sync;                       // null: plain kernel-to-kernel ordering
    int sync_signal;                 // != 0: this launch sets sync[0] and counts its stored tiles
    int sync_need;                   // > 0: this launch waits on sync[] instead of on the previous kernel
    // Grouped mode, optional: tiles are handed out in ascending order from this device counter (zeroed
    // by the caller) instead of in fixed strides, so that blocks which start late (the consuming
    // product's blocks reach an SM only when the producer's block there has left) or which drew long
    // tiles (uneven expert load) simply take fewer.
    int* tile_counter;
    int list_ready;                  // != 0: the tile list was complete before this kernel could start (the upstream
                                     // kernel lets its dependents go only after its own wait): no block-wide wait at the
                                     // top, set-up and weight prefetch overlap the upstream kernel
    int* status;                     // device status word (0 = ok)
    long long* trace;                // clock64 samples of block 0 in -DQMM_GEMM_TRACE=1 builds; unused (null) otherwise
};

// Pipeline geometry of one instantiation.  Tensor memory: half of the SM's 512 columns when the
// accumulators leave room for it (two blocks per SM), else all of it; what the accumulators leave
// is the weight ring.  A stage is one weight slot in TMEM plus one activation slot in shared memory.
template <int BN, int NA, int EPI, int FMT>
struct GemmGeom {
    static constexpr int kACols = NA * 32;                                 // TMEM columns per weight slot
    static constexpr int kDCols = NA * BN;                                 // accumulator columns
    static constexpr int kTmemCols = 512;                                  // all of it: one block per SM (registers)
    // two accumulator buffers (the epilogue of one piece overlaps the MMAs of the next) when a ring
    // of at least four weight slots still fits beside them
    static constexpr int kAccBufs = (2 * kDCols + 4 * kACols <= kTmemCols) ? 2 : 1;
    static constexpr int kFit = (kTmemCols - kAccBufs * kDCols) / kACols;
    static constexpr int kBStage = BN * kGemmBK * 2;                       // bytes per activation slot
    // the epilogue stages a finished tile in shared memory as fp16, [tile set][token pair][128 weight
    // rows] (32-bit words of two tokens): the outputs (plain store), or the gate and up accumulators
    // (SiLU*mul is applied on the way out)
    static constexpr int kStaging = NA * BN * 128 * 2;
    static constexpr int kSmemMax = 227 * 1024;                            // per block on sm_100
    static constexpr int kSmemFit = (kSmemMax - 1024 - 512 - kStaging) / kBStage;
    // With two weight tile sets tensor memory leaves a ring of three or four weight slots; an
    // activation tile takes ~1 800 cycles from the TMA request to its barrier, so a ring that shallow
    // for the activations bounds a stage at (MMA time + that latency) / slots.  The activation tiles
    // then get a ring of their own in shared memory with barriers of their own (kSplit), as deep as
    // shared memory allows; else one ring and one pair of barriers per stage serve both operands.
    // (also the 192-token tile with its two accumulator buffers: four weight slots.  Narrower tiles:
    // the extra waits and commits cost the issuing loop more than the latency they hide.)
    static constexpr bool kSplit = (NA == 2 && BN >= 128) || (NA == 1 && BN == 192);
    static constexpr int kFit2 = kSplit ? kFit : (kFit < kSmemFit ? kFit : kSmemFit);
    static constexpr int kStages = kFit2 < kGemmMaxStages ? kFit2 : kGemmMaxStages;             // weight slots (and activation slots unless kSplit)
    static constexpr int kStagesB = !kSplit ? kStages : (kSmemFit < kGemmMaxStagesB ? kSmemFit : kGemmMaxStagesB);
    static constexpr int kSmemBytes = kStagesB * kBStage + kStaging + 1024 /*align*/ + 512;
    // Warp roles: expanders, epilogue warps (one or two per TMEM lane quarter), TMA producer, MMA
    // issuer.  Narrow token tiles are bound by the expansion, not by the epilogue: 16 + 4 there,
    // and for two tile sets.
    // (two tile sets: every stage needs eight warp-stages of expansion, which eight warps do not
    // deliver in the 640 cycles of its MMAs)
    static constexpr bool kManyExpanders = BN <= 64 || NA == 2;
    // weight slices in flight per expander thread: one where there are 16 expander warps (each warp
    // then works on every second or fourth stage of its tile set, so its loads are as far ahead in
    // time as two slices with half the warps; measured 2-4 % faster for the 4-bit format, and the
    // 8-bit format's slices, twice the registers, only fit the 80 registers per thread this way)
    static constexpr int kPrefetch = kManyExpanders ? 1 : kGemmPrefetch;
    static constexpr int kExpWarps = kManyExpanders ? 16 : 8;
    static constexpr int kEpiWarps = kManyExpanders ? 4 : 8;
    // one MMA-issuing warp per weight tile set: each has its own accumulators, so nothing orders
    // their MMAs, and the loop that feeds the tensor pipe (the critical path with two tile sets: it
    // competes with four expander warps for its scheduler) runs in two halves side by side
    static constexpr int kIssuers = NA;
    static constexpr int kThreads = (kExpWarps + kEpiWarps + 1 + kIssuers) * 32;
    static_assert(kStages >= 2 && kStagesB >= 2, "tensor memory or shared memory over-subscribed");
};

// silu(g) = g / (1 + exp(-g)) with the fast exponential and reciprocal (relative error ~1e-6,
// far inside the fp16 rounding of the result; exp(-g) = inf for g < -88 gives -0, the right limit).
__device__ __forceinline__ float silu_f(float g) { return __fdividef(g, 1.0f + __expf(-g)); }

// One 64-k slice of a weight row as loaded (codes + scales), and its expansion
// to fp16(d * q) pairs, k ascending.  Loading and expanding are separate so
// that the loads of later slices can be in flight while one is expanded.
template <int FMT> struct RawRow64;
template <> struct RawRow64<QMM_Q4> {
    u32x8 c;
    uint32_t sc;
    __device__ __forceinline__ void load(const uint8_t* tile_ptr, int lane)
    {
        c = ld_keep_256(tile_ptr + 32 * lane);
        sc = ld_nc_u32(tile_ptr + kTileCodeBytes + 4 * lane);
    }
    __device__ __forceinline__ void expand(uint32_t (&out)[32], const Q4Consts& kc) const
    {
        const __half2 d0 = __half2half2(__low2half(as_h2(sc)));
        const __half2 d1 = __half2half2(__high2half(as_h2(sc)));
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            __half2 q[4];
            q4_word_to_h2(c.v[j], q, kc);
            const __half2 d = j < 4 ? d0 : d1;
#pragma unroll
            for (int p = 0; p < 4; ++p) out[4 * j + p] = as_u32(__hmul2(q[p], d));
        }
    }
};
// Q5 / Q6: the Q4 slice plus the row's high-bit words.
template <int FMT> struct RawRow64_56 {
    u32x8 c;
    uint32_t hi[Fmt<FMT>::hi_bytes / 4];
    uint32_t sc;
    __device__ __forceinline__ void load(const uint8_t* tile_ptr, int lane)
    {
        c = ld_keep_256(tile_ptr + 32 * lane);
#pragma unroll
        for (int i = 0; i < Fmt<FMT>::hi_bytes / 4; ++i) hi[i] = ld_nc_u32(tile_ptr + kTileCodeBytes + Fmt<FMT>::hi_bytes * lane + 4 * i);
        sc = ld_nc_u32(tile_ptr + Fmt<FMT>::scale_off + 4 * lane);
    }
    __device__ __forceinline__ void expand(uint32_t (&out)[32], const Q4Consts& kc) const
    {
        const __half2 d0 = __half2half2(__low2half(as_h2(sc)));
        const __half2 d1 = __half2half2(__high2half(as_h2(sc)));
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            __half2 q[4];
            q56_word_to_h2<FMT>(c.v[j], hi[FMT == QMM_Q5 ? j / 4 : j / 2], j, q, kc);
            const __half2 d = j < 4 ? d0 : d1;
#pragma unroll
            for (int p = 0; p < 4; ++p) out[4 * j + p] = as_u32(__hmul2(q[p], d));
        }
    }
};
template <> struct RawRow64<QMM_Q5> : RawRow64_56<QMM_Q5> {};
template <> struct RawRow64<QMM_Q6> : RawRow64_56<QMM_Q6> {};
template <> struct RawRow64<QMM_Q8> {
    u32x8 c[2];
    uint16_t sc[2];
    __device__ __forceinline__ void load(const uint8_t* tile_ptr, int lane)
    {
#pragma unroll
        for (int t = 0; t < 2; ++t) {                                     // two 32-k tiles
            const uint8_t* tp = tile_ptr + t * kQ8TileBytes;
            c[t] = ld_keep_256(tp + 32 * lane);
            sc[t] = ld_nc_u16(tp + kTileCodeBytes + 2 * lane);
        }
    }
    __device__ __forceinline__ void expand(uint32_t (&out)[32], const Q4Consts&) const
    {
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const __half2 d = __half2half2(__ushort_as_half(sc[t]));
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                __half2 q[2];
                q8_word_to_h2(c[t].v[j], q);
                out[16 * t + 2 * j] = as_u32(__hmul2(q[0], d));
                out[16 * t + 2 * j + 1] = as_u32(__hmul2(q[1], d));
            }
        }
    }
};

#ifndef QMM_GEMM_L2_AHEAD
#define QMM_GEMM_L2_AHEAD 6
#endif
// Clock samples of block 0's pipeline (tuning aid) exist only in builds with -DQMM_GEMM_TRACE=1: the
// shipped kernels carry no trace code.  The issuing loop's own samples need -DQMM_GEMM_TRACE_MMA=1 as
// well, because even a skipped sample costs the issuing warp instructions in its critical loop.
#ifndef QMM_GEMM_TRACE
#define QMM_GEMM_TRACE 0
#endif
#if QMM_GEMM_TRACE
#define QMM_TRACE_AT(cond, idx) \
    if (cond) p.trace[idx] = clock64();
#else
#define QMM_TRACE_AT(cond, idx)
#endif
#if QMM_GEMM_TRACE && defined(QMM_GEMM_TRACE_MMA) && QMM_GEMM_TRACE_MMA
#define QMM_TRACE_MMA(slot) \
    if (tracing && g + 1 < 64) p.trace[g * 8 + (slot)] = p.trace[(g + 1) * 8 + (slot)] = clock64();
#else
#define QMM_TRACE_MMA(slot)
#endif
constexpr int kGemmL2Ahead = QMM_GEMM_L2_AHEAD;    // stages of a row group's weight stream requested into L2 ahead of use

// One piece of work of a block: k-blocks [kb0, kb1) of one output tile.  `cn` blocks contribute to
// the tile (block indices first .. first + cn - 1, k ascending); cn == 1: the piece is the whole tile.
struct GemmWork {
    int n_tile, m_tile, expert, row0, rows;
    int n_mma;                       // token columns the MMAs of this piece compute: rows rounded up to 16
    int kb0, kb1;
    int first, cn;
};

// Epilogue of a piece of a tile that block boundaries cut (dense mode): store this warp's slice
// of the fp32 partial sums ([output tile][token column][128 weight rows]) and free the
// accumulators.  A second kernel adds the pieces of every cut tile in a fixed order.
template <int BN, int NOUT, int CH>
__device__ __noinline__ void cut_tile_epilogue(const GemmParams& p, const GemmWork& w, uint32_t lane_base, int quarter, int grp,
                                               int lane, uint64_t* acc_empty_bar)
{
    using namespace tc;
    constexpr size_t SLOT = (size_t)NOUT * BN * 128;                      // floats per partial slot
    // slot of this block's piece: 2 b + 1 for the piece that starts a tile, 2 b for one that continues it
    float* mine = p.partial + (size_t)(2 * blockIdx.x + ((int)blockIdx.x == w.first ? 1 : 0)) * SLOT + quarter * 32 + lane;
#pragma unroll 1
    for (int oc = 0; oc < NOUT * CH; ++oc) {
        const int o = oc / CH, c0 = (grp * CH + oc % CH) * 32;
        if (c0 < BN && c0 < w.rows) {
            uint32_t v[32];
            tmem_ld_32x32b_x32(lane_base + (uint32_t)(o * BN + c0), v);
            tmem_wait_ld();
            float* dst = mine + (size_t)(o * BN + c0) * 128;
#pragma unroll
            for (int j = 0; j < 32; ++j) __stcg(dst + j * 128, __uint_as_float(v[j]));
        }
    }
    tc_fence_before_sync();
    __syncwarp();
    if (lane == 0) mbar_arrive(acc_empty_bar);                            // the accumulators may be overwritten
}

// Persistent, warp-specialised kernel.  Tile t = (token tile t / n_tiles, weight
// tile t % n_tiles).  Grouped mode: every block walks the tile list t =
// blockIdx.x, blockIdx.x + gridDim.x, ... so blocks that run together share
// activation tiles.  Dense mode: every block takes the same number of whole
// tiles; the tiles that are left (all of them when there are few) are dealt
// either as equal contiguous shares of their (tile, k-block) units -- pieces
// of a tile cut by a share boundary go to fp32 partial sums -- or as half
// tiles of BN / 2 tokens, as the host's plan says.
// The pipeline (stage counter, barrier phases) runs on across pieces:
// while the epilogue warps drain the accumulators of piece i, the expanders
// and the TMA producer already fill the ring for piece i+1.
template <int FMT, int BN, int NA, int EPI, bool DENSE>
__global__ void __launch_bounds__(GemmGeom<BN, NA, EPI, FMT>::kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap x_map, const GemmParams p)
{
    using namespace tc;
    using G = GemmGeom<BN, NA, EPI, FMT>;
    constexpr int NEXP = G::kExpWarps;
    constexpr int PH = NEXP / (4 * NA);               // expander warps per (weight tile, lane quarter): they alternate stages
    constexpr int NEPI = G::kEpiWarps;
    constexpr int TMA_WARP = NEXP + NEPI, MMA_WARP = NEXP + NEPI + 1;   // issuers: warps MMA_WARP .. MMA_WARP + NISS - 1
    constexpr int NISS = G::kIssuers;
    constexpr int PREF = G::kPrefetch;                // weight slices in flight per expander thread
    constexpr int S = G::kStages;                     // pipeline depth (weight slots)
    constexpr bool SPLIT = G::kSplit;                 // activation tiles in a ring of their own
    constexpr int SB = G::kStagesB;                   // its depth (== S unless SPLIT)
    constexpr int A_COLS = G::kACols;
    constexpr int D_COLS = G::kDCols;
    constexpr int TMEM_COLS = G::kTmemCols;
    constexpr int AB = G::kAccBufs;                   // accumulator buffers: piece i uses buffer i % AB
    constexpr int RING0 = AB * D_COLS;                // first TMEM column of the weight ring
    static_assert(BN % 32 == 0 && BN >= 32 && BN <= 256, "token tile");
    static_assert(PH >= 1 && NEXP % 4 == 0, "expander warps must cover the four lane quarters");
    constexpr int B_STAGE = BN * kGemmBK * 2;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_b = smem;                                               // S slots, 1024-aligned each
    uint8_t* staging = smem + SB * B_STAGE;                               // finished tile, fp16 [output tile][token pair][128 rows]
    uint64_t* bars = reinterpret_cast<uint64_t*>(staging + G::kStaging);
    uint64_t* full = bars;                                                // [S] expanders + TMA -> MMA
    uint64_t* empty = bars + S;                                           // [S] MMA -> expanders, TMA
    uint64_t* acc_full = bars + 2 * S;                                    // [2] MMA -> epilogue
    uint64_t* acc_empty = bars + 2 * S + 2;                               // [2] epilogue -> MMA
    uint64_t* stg_full = bars + 2 * S + 4;                                // epilogue warps: tile staged
    uint64_t* stg_empty = bars + 2 * S + 5;                               // epilogue warps: staged tile stored
    uint64_t* full_b = bars + 2 * S + 6;                                  // [SB] TMA -> MMA          (SPLIT only)
    uint64_t* empty_b = bars + 2 * S + 6 + SB;                            // [SB] MMA -> TMA          (SPLIT only)
    uint64_t* seq_full = bars + 2 * S + 6 + 2 * SB;                       // [8] tile numbers drawn by the TMA lane (dynamic dealing)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 14 + 2 * SB);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* seq = reinterpret_cast<volatile int*>(tmem_slot + 2);   // [8]
    static_assert((2 * S + 14 + 2 * SB) * 8 + 8 + 32 <= 512, "barrier area");

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr bool grouped = !DENSE;                                      // token tiles come from a device-built list
    // the tile list is written upstream: wait for the previous kernel, or (hand-over by tiles) for the
    // flag that the producing product sets once its own wait for the upstream kernels has returned
    const bool by_tiles = grouped && p.sync != nullptr && p.sync_need > 0;
    if (grouped && !by_tiles && !p.list_ready) {
        pdl_wait();
        if (p.sync != nullptr && p.sync_signal && blockIdx.x == 0 && threadIdx.x == 0) {
            __threadfence();
            atomicExch(p.sync, 1);
        }
    }
    if (by_tiles) {
        __shared__ int s_list_ok;
        if (threadIdx.x == 0) {
            const long long t0 = clock64();
            int ok = 1;
            while (*reinterpret_cast<volatile int*>(p.sync) == 0) {
                if (clock64() - t0 > tc::kWaitLimitCycles) {
                    ok = 0;
                    break;
                }
            }
            __threadfence();
            s_list_ok = ok;
        }
        __syncthreads();
        if (!s_list_ok) {                                                 // nothing is allocated or in flight yet
            if (threadIdx.x == 0 && p.status != nullptr) atomicExch(p.status, (int)QMM_ERR_DEVICE_TIMEOUT);
            return;
        }
    }
    // plain store: the NA tile sets split the rows of one matrix; SiLU*mul: they are two matrices of N rows each
    const int n_tiles = (EPI == kEpiSiluMul) ? p.N / 128 : p.N / (128 * NA);
    const int m_tiles = grouped ? *p.num_tiles : (p.M + BN - 1) / BN;
    const int total_tiles = n_tiles * m_tiles;
    const int KB = p.K / kGemmBK;                                         // k-blocks per tile
    const int U = DENSE && !grouped ? p.units_per_block : 0;           // (a compile-time 0 in the grouped kernels)

    // ---- set-up
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full[s], 4 * NA + (SPLIT ? 0 : 1));                // the stage's expander warps (+ the TMA producer)
            mbar_init(&empty[s], NISS);                                   // one tcgen05.commit per issuing warp
        }
        if (SPLIT)
            for (int s = 0; s < SB; ++s) {
                mbar_init(&full_b[s], 1);                                 // the TMA producer (+ its bytes)
                mbar_init(&empty_b[s], NISS);                             // one tcgen05.commit per issuing warp
            }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&acc_full[b], NISS);
            mbar_init(&acc_empty[b], NEPI);
        }
        mbar_init(stg_full, NEPI);
        mbar_init(stg_empty, NEPI);
        for (int q = 0; q < 8; ++q) mbar_init(&seq_full[q], 1);
        *abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == MMA_WARP) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    if (warp == TMA_WARP && lane == 0) prefetch_tensormap(&x_map);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    pdl_launch_dependents();

    // i-th piece of work of this block (every role walks the same sequence); false past the last
    auto get_work = [&](int i, GemmWork& w) -> bool {
        int t;
        int half = -1;                                                    // >= 0: which half of the tile's tokens
        const int whole = DENSE ? p.whole_tiles / (int)gridDim.x : 0;     // whole tiles of this block, taken first
        if (DENSE && i >= whole && p.tail_halves) {
            // the tiles of the last, partly filled round as half tiles (no partial sums: each half is a
            // product of its own; its weights are expanded twice)
            const int j = (int)blockIdx.x + (i - whole) * (int)gridDim.x;
            if (j >= 2 * (total_tiles - p.whole_tiles)) return false;
            t = p.whole_tiles + (j >> 1);
            half = j & 1;
            w.kb0 = 0;
            w.kb1 = KB;
            w.first = blockIdx.x;
            w.cn = 1;
        } else if (DENSE && i < whole) {
            t = (int)blockIdx.x * whole + i;
            w.kb0 = 0;
            w.kb1 = KB;
            w.first = blockIdx.x;
            w.cn = 1;
        } else if (U > 0) {
            i -= whole;
            const int t0 = DENSE ? p.whole_tiles : 0;                     // the tiles below are counted from here
            const long long u0 = (long long)blockIdx.x * U;
            const long long u1 = min(u0 + U, (long long)(total_tiles - t0) * KB);
            if (u0 >= u1) return false;
            // Tiles the share touches: first .. last.  Order of work: the cut tile at the head of the
            // share, the cut tile at its tail, then the whole tiles -- cut tiles are then completed
            // (by this block or a neighbour) while whole tiles are still being computed.
            const int t_first = (int)(u0 / KB), t_last = (int)((u1 - 1) / KB);
            if (i > t_last - t_first) return false;
            const int hc = u0 > (long long)t_first * KB ? 1 : 0;
            const int tc = (t_last > t_first && u1 < (long long)(t_last + 1) * KB) ? 1 : 0;
            if (hc && i == 0) t = t_first;
            else if (tc && i == hc) t = t_last;
            else t = t_first + i - tc;
            const long long tb = (long long)t * KB;                       // first unit of tile t
            w.kb0 = (int)max(u0 - tb, 0LL);
            w.kb1 = (int)min(u1 - tb, (long long)KB);
            const int Ud = U > 0 ? U : 1;                                 // (U > 0 here; spelled out for the grouped instantiations)
            w.first = (int)(tb / Ud);
            w.cn = (int)((tb + KB - 1) / Ud) - w.first + 1;
            t += t0;
        } else {
            if (grouped && p.tile_counter != nullptr) {
                // the TMA lane draws the block's i-th tile and publishes it to the other roles through a
                // small ring (no role is ever more than a few tiles ahead of the epilogue, far fewer than 8)
                const int slot = i & 7;
                if (warp == TMA_WARP) {
                    t = atomicAdd(p.tile_counter, 1);
                    seq[slot] = t;
                    mbar_arrive(&seq_full[slot]);
                } else {
                    if (!mbar_wait(&seq_full[slot], (i >> 3) & 1, abort_flag)) return false;
                    t = seq[slot];
                }
            } else {
                t = blockIdx.x + i * gridDim.x;
            }
            if (t >= total_tiles) return false;
            w.kb0 = 0;
            w.kb1 = KB;
            w.first = blockIdx.x;
            w.cn = 1;
        }
        w.n_tile = t % n_tiles;
        const int mt = t / n_tiles;
        w.m_tile = mt;
        if (grouped) {
            w.expert = p.tile_expert[mt];
            w.row0 = p.tile_row0[mt];
            w.rows = p.tile_rows[mt];
        } else {
            w.expert = 0;
            w.row0 = mt * BN;
            w.rows = min(BN, p.M - w.row0);
        }
        if (DENSE && half >= 0) {
            w.row0 += half * (BN / 2);
            w.rows = max(0, min(BN / 2, p.M - w.row0));
        }
        w.n_mma = max(16, min(BN, (w.rows + 15) & ~15));                  // valid rows rounded up to the MMA's granularity
        return true;
    };

    if (warp < NEXP) {
        // ================= expanders: weights -> fp16 -> TMEM A ring
        const int quarter = warp & 3;                                     // TMEM lane quarter
        const int a = (warp >> 2) % NA;                                   // weight tile set
        const int phase = (warp >> 2) / NA;                               // takes the stages g = phase (mod PH)
        const int tpr = p.K / Fmt<FMT>::tile_k;
        constexpr int TILES_PER_KB = kGemmBK / Fmt<FMT>::tile_k;
        const size_t kb_bytes = (size_t)TILES_PER_KB * Fmt<FMT>::tile_bytes;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const uint8_t* wmat = (NA == 2 && a == 1) ? p.w[1] : p.w[0];      // (not p.w[a]: indexing a kernel parameter by a run-time value copies the parameters to local memory)
        Q4Consts kc;
        kc.init();
        bool ok = true;
        int g0 = 0;                                                       // stage counter at the start of the piece
        GemmWork w;
        for (int i = 0; ok && get_work(i, w); ++i) {
            const int num_kb = w.kb1 - w.kb0;
            const int rg = w.n_tile * 4 + quarter;                        // row group of 32 rows
            const uint8_t* wrow = wmat + (size_t)w.expert * p.w_expert_stride + (size_t)rg * tpr * Fmt<FMT>::tile_bytes +
                                  (size_t)w.kb0 * kb_bytes;                // this piece's part of the row group's stream
            // The weight stream of a row group is contiguous: ask L2 for it kGemmL2Ahead stages ahead
            // (expert weights come from HBM; two register-held slices alone do not cover that latency).
            if (lane == 0 && phase == 0) {
                const int ahead = num_kb < kGemmL2Ahead ? num_kb : kGemmL2Ahead;
                l2_prefetch(wrow, (uint32_t)(ahead * kb_bytes));
            }
            RawRow64<FMT> raw[PREF];
#pragma unroll
            for (int i = 0; i < PREF; ++i)
                if (phase + i * PH < num_kb) raw[i].load(wrow + (size_t)(phase + i * PH) * kb_bytes, lane);
            for (int kb0 = phase; kb0 < num_kb && ok; kb0 += PREF * PH) {
#pragma unroll
                for (int i = 0; i < PREF; ++i) {
                    const int kb = kb0 + i * PH;
                    if (kb >= num_kb || !ok) break;
                    const int g = g0 + kb;
                    const int s = g % S;
                    uint32_t vals[32];
                    [[maybe_unused]] const bool tr = QMM_GEMM_TRACE && p.trace != nullptr && blockIdx.x == 0 && g < 64 && quarter == 0 && a == 0 && lane == 0;
                    QMM_TRACE_AT(tr, g * 8 + 4)
                    raw[i].expand(vals, kc);
                    if (kb + PREF * PH < num_kb) raw[i].load(wrow + (size_t)(kb + PREF * PH) * kb_bytes, lane);
                    if (lane == 0 && kb + kGemmL2Ahead < num_kb) l2_prefetch(wrow + (size_t)(kb + kGemmL2Ahead) * kb_bytes, (uint32_t)kb_bytes);
                    QMM_TRACE_AT(tr, g * 8 + 5)
                    QMM_TRACE_AT(tr, g * 8 + 6)
                    if (g >= S) ok = mbar_wait(&empty[s], ((g / S) - 1) & 1, abort_flag);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after_sync();
                    QMM_TRACE_AT(tr, g * 8 + 7)
                    tmem_st_32x32b_x32(lane_base + (uint32_t)(RING0 + s * A_COLS + a * 32), vals);
                    // announce the slot at once: deferring the wait for the store behind the next
                    // expansion was measured and costs more in slot turn-around than the ~85 cycles it hides
                    tmem_wait_st();
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&full[s]);
                }
            }
            g0 += num_kb;
        }
        if (!ok) *abort_flag = 1;
    } else if (warp < NEXP + NEPI) {
        // ================= epilogue: TMEM -> registers -> global
        const int e = warp - NEXP;
        const int quarter = e & 3;                                        // == warp & 3: the lanes this warp may read
        constexpr int GROUPS = NEPI / 4;                                  // warps per lane quarter: they split the token columns
        const int grp = e >> 2;
        uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);   // + the piece's accumulator buffer
        int buf = 0;
        constexpr int NCH = BN / 32;                                      // 32-column chunks of the tile
        constexpr int CH = (NCH + GROUPS - 1) / GROUPS;                   // chunks per warp
        constexpr int NOUT = (EPI == kEpiSiluMul) ? 1 : NA;               // output tiles per weight row
        constexpr int NSTG = NA;                                          // tile sets that go through the staging buffer
        if (!by_tiles) pdl_wait();                                        // the output buffer may be in use upstream
        bool ok = true;
        [[maybe_unused]] bool etr = false;
        int it = 0, staged = 0;                                           // pieces seen / tiles that went through the staging buffer
        const uint32_t stg_lane = smem_u32(staging) + (uint32_t)((quarter * 32 + lane) * 4);   // this thread's weight row
        // 32 tokens (one chunk) of this thread's weight row -> staging[o][(c0 + 2j) / 2][row] as fp16
        // pairs (tokens 2j, 2j+1 of one weight row share a 32-bit word: one store per converted pair)
        auto stage_chunk = [&](int o, int c0, const uint32_t (&v)[32]) {
            const uint32_t dst = stg_lane + (uint32_t)(((o * BN + c0) >> 1) * 512);
#pragma unroll
            for (int j = 0; j < 16; ++j)
                st_shared_b32(dst + (uint32_t)(j * 512),
                              as_u32(__floats2half2_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1]))));
        };
        auto release = [&]() {                                            // the next piece may overwrite the accumulators
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
            QMM_TRACE_AT(etr, (it * 4 + 2) * 8 + 1)
        };
        GemmWork w;
        for (; ok && get_work(it, w); ++it) {
            const int rows = w.rows;
            buf = it % AB;
            lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * D_COLS);
            ok = mbar_wait(&acc_full[buf], (it / AB) & 1, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            etr = QMM_GEMM_TRACE && p.trace != nullptr && blockIdx.x == 0 && it < 16 && e == 0 && lane == 0;
            QMM_TRACE_AT(etr, (it * 4 + 1) * 8 + 1)
            if (DENSE && w.cn > 1) {
                // a tile cut by block boundaries (dense mode only): out of line, so that its registers
                // do not weigh on the common path
                if constexpr (DENSE) cut_tile_epilogue<BN, NOUT, CH>(p, w, lane_base, quarter, grp, lane, &acc_empty[buf]);
                continue;
            }
            if (staged > 0) {                                             // the previous staged tile must have been stored
                ok = mbar_wait(stg_empty, (staged - 1) & 1, abort_flag);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
            }
            {
                // (SiLU*mul: the gate and up accumulators are staged as fp16 and combined when the tile
                // is stored, after the accumulators have been handed back)
                // two chunk loads in flight per wait (an invalid second chunk re-reads the first and is dropped)
#pragma unroll
                for (int o = 0; o < NSTG; ++o) {
#pragma unroll
                    for (int c = 0; c < CH; c += 2) {
                        const int c0 = (grp * CH + c) * 32, c1 = c0 + 32;
                        const bool v0 = c0 < BN && c0 < rows, v1 = c + 1 < CH && c1 < BN && c1 < rows;
                        if (v0) {
                            uint32_t va[32], vb[32];
                            tmem_ld_32x32b_x32(lane_base + (uint32_t)(o * BN + c0), va);
                            tmem_ld_32x32b_x32(lane_base + (uint32_t)(o * BN + (v1 ? c1 : c0)), vb);
                            tmem_wait_ld();
                            stage_chunk(o, c0, va);
                            if (v1) stage_chunk(o, c1, vb);
                        }
                    }
                }
            }
            release();
            // all eight warps staged -> store the tile: two token rows (2 x 256 bytes) per warp instruction
            __syncwarp();
            if (lane == 0) mbar_arrive(stg_full);
            ok = mbar_wait(stg_full, staged & 1, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            if constexpr (EPI == kEpiSiluMul) {
                // two token rows per warp instruction: a lane combines the gate and up values of its 4
                // weight rows for tokens 2 rp, 2 rp + 1 (one 16-byte read each) and stores 8 bytes per row
                uint16_t* out = p.out + (size_t)w.row0 * p.ldo + (size_t)w.n_tile * 128 + lane * 4;
                const uint32_t src = smem_u32(staging) + (uint32_t)(lane * 16);
                auto silu_mul = [](uint32_t g, uint32_t u, float& lo, float& hi) {    // words of two tokens
                    const float2 gf = __half22float2(as_h2(g)), uf = __half22float2(as_h2(u));
                    lo = silu_f(gf.x) * uf.x;
                    hi = silu_f(gf.y) * uf.y;
                };
                for (int rp = e; 2 * rp < rows; rp += NEPI) {
                    const uint4 g = ld_shared_v4(src + (uint32_t)(rp * 512));
                    const uint4 u = ld_shared_v4(src + (uint32_t)(((BN >> 1) + rp) * 512));
                    float a0, b0, a1, b1, a2, b2, a3, b3;                 // a: token 2 rp, b: token 2 rp + 1
                    silu_mul(g.x, u.x, a0, b0);
                    silu_mul(g.y, u.y, a1, b1);
                    silu_mul(g.z, u.z, a2, b2);
                    silu_mul(g.w, u.w, a3, b3);
                    uint2 h;
                    h.x = as_u32(__floats2half2_rn(a0, a1));
                    h.y = as_u32(__floats2half2_rn(a2, a3));
                    *reinterpret_cast<uint2*>(out + (size_t)(2 * rp) * p.ldo) = h;
                    if (2 * rp + 1 < rows) {
                        h.x = as_u32(__floats2half2_rn(b0, b1));
                        h.y = as_u32(__floats2half2_rn(b2, b3));
                        *reinterpret_cast<uint2*>(out + (size_t)(2 * rp + 1) * p.ldo) = h;
                    }
                }
            } else {
                // lanes 0-15: token row r, lanes 16-31: row r + 1 (the same staged words, the other half);
                // a lane gathers the 8 weight rows of its 16-byte output segment from 8 words
                const int half = lane >> 4, seg = lane & 15;
                uint16_t* out = p.out + (size_t)w.row0 * p.ldo + (size_t)w.n_tile * 128 + seg * 8;
                const uint32_t src = smem_u32(staging) + (uint32_t)(seg * 32);
                const uint32_t sel = half ? 0x7632u : 0x5410u;            // high / low fp16 of two words
#pragma unroll
                for (int o = 0; o < NOUT; ++o) {
                    for (int r = 2 * e + half; r < rows; r += 2 * NEPI) {
                        const uint32_t a = src + (uint32_t)(((o * BN + r) >> 1) * 512);
                        const uint4 w0 = ld_shared_v4(a), w1 = ld_shared_v4(a + 16);
                        uint4 v;
                        v.x = __byte_perm(w0.x, w0.y, sel);
                        v.y = __byte_perm(w0.z, w0.w, sel);
                        v.z = __byte_perm(w1.x, w1.y, sel);
                        v.w = __byte_perm(w1.z, w1.w, sel);
                        *reinterpret_cast<uint4*>(out + (size_t)r * p.ldo + (size_t)o * p.a_col_offset) = v;
                    }
                }
            }
            if (grouped && p.sync != nullptr && p.sync_signal) {          // this warp's part of the token tile is stored
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(p.sync + 1 + w.m_tile, 1);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(stg_empty);
            ++staged;
        }
        if (!ok) *abort_flag = 1;
    } else if (warp == TMA_WARP) {
        // ================= TMA producer: activation tiles
        if (lane == 0) {
            if (!by_tiles) pdl_wait();                                    // activations come from the previous kernel
            if (grouped && p.list_ready && p.sync != nullptr && p.sync_signal && blockIdx.x == 0) {
                __threadfence();                                          // everything upstream is complete: the consuming product may read the list
                atomicExch(p.sync, 1);
            }
            int issued = 0, g = 0;
            bool ok = true;
            GemmWork w;
            for (int i = 0; ok && get_work(i, w); ++i) {
                if (by_tiles) {
                    // the rows of this token tile are complete once every epilogue warp of the producing
                    // product has counted itself in for each of its weight tiles
                    const volatile int* cnt = p.sync + 1 + w.m_tile;
                    const long long t0 = clock64();
                    while (*cnt < p.sync_need) {
                        if (*abort_flag || clock64() - t0 > tc::kWaitLimitCycles) {
                            ok = false;
                            break;
                        }
                    }
                    if (!ok) break;
                    __threadfence();
                    asm volatile("fence.proxy.async;" ::: "memory");     // the rows were written by ordinary stores, TMA reads them
                }
                for (int kb = w.kb0; kb < w.kb1; ++kb, ++g) {
                    const int s = g % SB;
                    uint64_t* slot_full = SPLIT ? &full_b[s] : &full[s];
                    if (g >= SB) ok = mbar_wait(SPLIT ? &empty_b[s] : &empty[s], ((g / SB) - 1) & 1, abort_flag);
                    if (!ok) break;
                    mbar_arrive_expect_tx(slot_full, B_STAGE);
                    tma_load_2d(smem_b + s * B_STAGE, &x_map, kb * kGemmBK, w.row0, slot_full);
                    issued = g + 1;
                }
            }
            if (!ok) {
                *abort_flag = 1;
                // let loads in flight land before the block's shared memory is released
                // (the same barrier also counts expander arrivals, so this can run into its time limit)
                for (int q = max(0, issued - SB); q < issued; ++q) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(SPLIT ? &full_b[q % SB] : &full[q % S], (q / SB) & 1) && clock64() - t0 < (1LL << 22)) {}
                }
            }
        }
    } else {
        // ================= MMA issuer
        // The whole warp runs the loop converged (so that addresses and descriptors stay warp-uniform
        // values); one elected lane issues the MMAs and the commits.
        const uint64_t desc0 = smem_desc_k_sw128(smem_u32(smem_b));       // slot 0, k-step 0
        const int ia = warp - MMA_WARP;                                   // which issuer
        bool ok = true;
        int g = 0, it = 0;
        // The issuing lane.  The MMAs and commits below are predicated on it instead of sitting in a
        // divergent branch: measured ~25 % less issue time per stage (operands stay warp-uniform).
        const uint32_t sel = elect_one() ? 1u : 0u;
        [[maybe_unused]] const bool tracing = QMM_GEMM_TRACE && p.trace != nullptr && blockIdx.x == 0 && lane == 0 && warp == MMA_WARP;
        (void)g;
        int s = 0;                                                        // ring slot of stage g and the parity of its
        uint32_t par = 0;                                                 // "full" barrier, carried across pieces
        int sb = 0;                                                       // the same for the activation ring (SPLIT)
        uint32_t parb = 0;
        GemmWork w;
        for (; ok && get_work(it, w); ++it) {
            const int buf = it % AB;
            if (it >= AB) {                                               // the epilogue must have read this buffer's previous piece
                ok = mbar_wait(&acc_empty[buf], ((it / AB) - 1) & 1, abort_flag);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after_sync();
                QMM_TRACE_AT(tracing && it <= 16, ((it - AB) * 4 + 3) * 8 + 1)
            }
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * D_COLS);
            // The MMAs' N is the piece's valid token rows rounded up to 16 (a partly filled expert tile,
            // the ragged last token tile of a dense product, a half tile of its last round): the tensor
            // time shrinks with it, and the columns beyond are never read.
            const uint32_t idesc = idesc_f16_m128(w.n_mma);
            // One round of the loop = wait for the slot(s), vote, fence, MMAs, commit(s).  Two stages per
            // round when the ring is deep enough (the polls, the vote and the fence are paid once per
            // 128 k), then single stages for what is left of the piece.  Both bodies are straight-line
            // code: a common body with a run-time stage count per round was measured at ~100 cycles more
            // per stage in the issuing warp, which the short MMA queue does not hide.
            static_assert(kGemmBK == 64, "four K = 16 steps per stage");
            // MMAs of stage kb from ring slot sj (descriptor start address is in 16-byte units: slot s is
            // s * B_STAGE / 16 further), then the commit that frees the slot
            auto issue_stage = [&](int sj, bool acc) {
                const uint64_t desc_s = desc0 + (uint64_t)((SPLIT ? sb : sj) * (B_STAGE >> 4));
                const uint32_t a_s = tmem_base + (uint32_t)(RING0 + sj * A_COLS);
#pragma unroll
                for (int a = 0; a < NA / NISS; ++a)                       // this warp's tile set(s)
                    mma_ts_f16_stage(d_tmem + (uint32_t)((ia + a * NISS) * BN), a_s + (uint32_t)((ia + a * NISS) * 32), desc_s, idesc, acc, sel);
                mma_commit_sel(&empty[sj], sel);                          // slot reusable when these MMAs finish
                if constexpr (SPLIT) mma_commit_sel(&empty_b[sb], sel);
            };
            auto next_b = [&]() {                                         // advance the activation ring (SPLIT)
                if (++sb == SB) {
                    sb = 0;
                    parb ^= 1;
                }
            };
            int kb = w.kb0;
            if constexpr (S >= 6) {
                for (; kb + 2 <= w.kb1 && ok; kb += 2) {
                    int s1 = s + 1;
                    uint32_t par1 = par;
                    if (s1 == S) {
                        s1 = 0;
                        par1 ^= 1;
                    }
                    QMM_TRACE_MMA(0)
                    ok = mbar_wait(&full[s], par, abort_flag);
                    if (ok) ok = mbar_wait(&full[s1], par1, abort_flag);
                    if constexpr (SPLIT) {
                        int sb1 = sb + 1;
                        uint32_t parb1 = parb;
                        if (sb1 == SB) {
                            sb1 = 0;
                            parb1 ^= 1;
                        }
                        if (ok) ok = mbar_wait(&full_b[sb], parb, abort_flag);
                        if (ok) ok = mbar_wait(&full_b[sb1], parb1, abort_flag);
                    }
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    QMM_TRACE_MMA(2)
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_stage(s, kb != w.kb0);
                    if constexpr (SPLIT) next_b();
                    issue_stage(s1, true);
                    if constexpr (SPLIT) next_b();
                    __syncwarp();
                    QMM_TRACE_MMA(3)
                    g += 2;
                    s = s1 + 1;
                    par = par1;
                    if (s == S) {
                        s = 0;
                        par ^= 1;
                    }
                }
            }
            for (; kb < w.kb1 && ok; ++kb) {
                QMM_TRACE_MMA(0)
                ok = mbar_wait(&full[s], par, abort_flag);
                if constexpr (SPLIT) {
                    if (ok) ok = mbar_wait(&full_b[sb], parb, abort_flag);
                }
                ok = __all_sync(0xFFFFFFFFu, ok);
                QMM_TRACE_MMA(2)
                if (!ok) break;
                tc_fence_after_sync();
                issue_stage(s, kb != w.kb0);
                __syncwarp();
                QMM_TRACE_MMA(3)
                ++g;
                if (++s == S) {
                    s = 0;
                    par ^= 1;
                }
                if constexpr (SPLIT) next_b();
            }
            if (ok) mma_commit_sel(&acc_full[buf], sel);                  // accumulators of this piece are complete
            __syncwarp();
            QMM_TRACE_AT(tracing && it < 16, (it * 4 + 0) * 8 + 1)
        }
        if (!ok) *abort_flag = 1;
    }

    // ---- teardown
    tc_fence_before_sync();
    __syncthreads();
    if (threadIdx.x == 0 && *abort_flag && p.status != nullptr) atomicExch(p.status, (int)QMM_ERR_DEVICE_TIMEOUT);
    if (warp == MMA_WARP) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace qmm
