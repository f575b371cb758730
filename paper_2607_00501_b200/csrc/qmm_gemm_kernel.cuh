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
//   expanders (8 warps): 8 / (4*NA) per weight tile and lane quarter,
//                      alternating stages; thread = one weight row; 32-byte
//                      code loads straight from global/L2, unpack to fp16(d*q),
//                      tcgen05.st into the A ring in TMEM.
//   epilogue (8 warps, two per lane quarter): tcgen05.ld the accumulators,
//                      release them, store fp16.
//   TMA producer (1 warp): activation tiles -> shared-memory ring (128-byte
//                      swizzle), one elected lane.
//   MMA issuer (1 warp, converged): one elected lane issues tcgen05.mma
//                      (M128 x N=BN x K16), frees ring slots with tcgen05.commit.
// The kernel is persistent: a block loops over tiles and the pipeline runs on
// across tile boundaries.
//
// TMEM columns: [0, NA*BN) fp32 accumulators, then STAGES slots of NA*32
// columns (64 fp16 k-values per row and weight tile).
//
// Every mbarrier wait is bounded; on give-up the block raises an abort flag,
// records QMM_ERR_DEVICE_TIMEOUT in the status word, stops issuing work, waits
// (bounded) for its outstanding TMA loads, frees its TMEM and returns.
#pragma once

#include "qmm_common.cuh"
#include "qmm_tc.cuh"

namespace qmm {

constexpr int kGemmBK = 64;          // k per pipeline stage
constexpr int kGemmMaxStages = 6;     // pipeline depth is min(this, what tensor memory leaves for the weight ring)

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
    int splits;                      // K splits (dense only, >= 1): > 1 -> fp32 partial sums go to `partial`
    float* partial;                  // [splits][M][N-wide rows] fp32, when splits > 1
    int* status;                     // device status word (0 = ok)
    long long* trace;                // optional [block 0 only] clock64 samples for pipeline analysis (tuning aid), else null
};

// Pipeline geometry of one instantiation.  Tensor memory: half of the SM's 512 columns when the
// accumulators leave room for it (two blocks per SM), else all of it; what the accumulators leave
// is the weight ring.  A stage is one weight slot in TMEM plus one activation slot in shared memory.
template <int BN, int NA>
struct GemmGeom {
    static constexpr int kACols = NA * 32;                                 // TMEM columns per weight slot
    static constexpr int kDCols = NA * BN;                                 // accumulator columns
    static constexpr int kTmemCols = kDCols <= 128 ? 256 : 512;
    static constexpr int kFit = (kTmemCols - kDCols) / kACols;
    static constexpr int kStages = kFit < kGemmMaxStages ? kFit : kGemmMaxStages;
    static constexpr int kBStage = BN * kGemmBK * 2;                       // bytes per activation slot
    static constexpr int kSmemBytes = kStages * kBStage + 1024 /*align*/ + 256;
    // Warp roles: 8 expanders, 8 epilogue warps (two per TMEM lane quarter), TMA producer, MMA issuer.
    static constexpr int kExpWarps = 8;
    static constexpr int kEpiWarps = 8;
    static constexpr int kThreads = (kExpWarps + kEpiWarps + 2) * 32;
    static_assert(kStages >= 2, "tensor memory over-subscribed");
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

constexpr int kGemmPrefetch = 2;     // weight slices in flight per expander thread
constexpr int kGemmL2Ahead = 12;     // stages of a row group's weight stream requested into L2 ahead of use

// Persistent, warp-specialised kernel.  Every block walks the tile list
// t = blockIdx.x, blockIdx.x + gridDim.x, ...; tile t = (token tile t / n_tiles,
// weight tile t % n_tiles), so blocks that run together share activation tiles.
// The pipeline (stage counter, barrier phases) runs on across tiles: while the
// epilogue warps drain the accumulators of tile i, the expanders and the TMA
// producer already fill the ring for tile i+1.
template <int FMT, int BN, int NA, int EPI>
__global__ void __launch_bounds__(GemmGeom<BN, NA>::kThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap x_map, const GemmParams p)
{
    using namespace tc;
    using G = GemmGeom<BN, NA>;
    constexpr int NEXP = G::kExpWarps;
    constexpr int PH = NEXP / (4 * NA);               // expander warps per (weight tile, lane quarter): they alternate stages
    constexpr int NEPI = G::kEpiWarps;
    constexpr int TMA_WARP = NEXP + NEPI, MMA_WARP = NEXP + NEPI + 1;
    constexpr int S = G::kStages;                     // pipeline depth
    constexpr int A_COLS = G::kACols;
    constexpr int D_COLS = G::kDCols;
    constexpr int TMEM_COLS = G::kTmemCols;
    static_assert(BN % 32 == 0 && BN >= 32 && BN <= 256, "token tile");
    static_assert(PH >= 1 && NEXP % 4 == 0, "expander warps must cover the four lane quarters");
    constexpr int B_STAGE = BN * kGemmBK * 2;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* smem_b = smem;                                               // S slots, 1024-aligned each
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + S * B_STAGE);
    uint64_t* full = bars;                                                // [S] expanders + TMA -> MMA
    uint64_t* empty = bars + S;                                           // [S] MMA -> expanders, TMA
    uint64_t* acc_full = bars + 2 * S;                                    // MMA -> epilogue
    uint64_t* acc_empty = bars + 2 * S + 1;                               // epilogue -> MMA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const bool grouped = p.tile_expert != nullptr;
    if (grouped) pdl_wait();                                              // the tile list is written upstream
    // plain store: the NA tile sets split the rows of one matrix; SiLU*mul: they are two matrices of N rows each
    const int n_tiles = (EPI == kEpiSiluMul) ? p.N / 128 : p.N / (128 * NA);
    const int m_tiles = grouped ? *p.num_tiles : (p.M + BN - 1) / BN;
    const int splits = grouped || p.splits < 1 ? 1 : p.splits;           // K splits: a tile is (token tile, weight tile, split)
    const int total_tiles = n_tiles * m_tiles * splits;
    const int num_kb = p.K / kGemmBK / splits;                            // k-blocks per tile

    // ---- set-up
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) {
            mbar_init(&full[s], 4 * NA + 1);                              // the stage's expander warps + the TMA producer
            mbar_init(&empty[s], 1);                                      // one tcgen05.commit
        }
        mbar_init(acc_full, 1);
        mbar_init(acc_empty, NEPI);
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

    // token rows of tile t
    auto tile_rows = [&](int t, int& n_tile, int& expert, int& row0, int& rows, int& ks) {
        ks = t % splits;
        t /= splits;
        n_tile = t % n_tiles;
        const int mt = t / n_tiles;
        if (grouped) {
            expert = p.tile_expert[mt];
            row0 = p.tile_row0[mt];
            rows = p.tile_rows[mt];
        } else {
            expert = 0;
            row0 = mt * BN;
            rows = min(BN, p.M - row0);
        }
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
        Q4Consts kc;
        kc.init();
        bool ok = true;
        int pending = -1;                                                 // stage stored but not yet announced
        // The store of one stage is announced (wait::st + arrive) only after the next stage has been
        // expanded, so the tensor-memory write latency hides behind ALU work.
        auto announce = [&]() {
            if (pending >= 0) {
                tmem_wait_st();
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive(&full[pending]);
                pending = -1;
            }
        };
        int g0 = 0;                                                       // stage counter at the start of the tile
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, g0 += num_kb) {
            int n_tile, expert, row0, rows, ks;
            tile_rows(t, n_tile, expert, row0, rows, ks);
            const int rg = n_tile * 4 + quarter;                          // row group of 32 rows
            const uint8_t* wrow = p.w[a] + (size_t)expert * p.w_expert_stride + (size_t)rg * tpr * Fmt<FMT>::tile_bytes +
                                  (size_t)ks * num_kb * kb_bytes;          // this split's part of the row group's stream
            // The weight stream of a row group is contiguous: ask L2 for it kGemmL2Ahead stages ahead
            // (expert weights come from HBM; two register-held slices alone do not cover that latency).
            if (lane == 0 && phase == 0) {
                const int ahead = num_kb < kGemmL2Ahead ? num_kb : kGemmL2Ahead;
                l2_prefetch(wrow, (uint32_t)(ahead * kb_bytes));
            }
            RawRow64<FMT> raw[kGemmPrefetch];
#pragma unroll
            for (int i = 0; i < kGemmPrefetch; ++i)
                if (phase + i * PH < num_kb) raw[i].load(wrow + (size_t)(phase + i * PH) * kb_bytes, lane);
            for (int kb0 = phase; kb0 < num_kb && ok; kb0 += kGemmPrefetch * PH) {
#pragma unroll
                for (int i = 0; i < kGemmPrefetch; ++i) {
                    const int kb = kb0 + i * PH;
                    if (kb >= num_kb || !ok) break;
                    const int g = g0 + kb;
                    const int s = g % S;
                    uint32_t vals[32];
                    const bool tr = p.trace != nullptr && blockIdx.x == 0 && g < 64 && quarter == 0 && a == 0 && lane == 0;
                    if (tr) p.trace[g * 8 + 4] = clock64();
                    raw[i].expand(vals, kc);
                    if (kb + kGemmPrefetch * PH < num_kb) raw[i].load(wrow + (size_t)(kb + kGemmPrefetch * PH) * kb_bytes, lane);
                    if (lane == 0 && kb + kGemmL2Ahead < num_kb) l2_prefetch(wrow + (size_t)(kb + kGemmL2Ahead) * kb_bytes, (uint32_t)kb_bytes);
                    if (tr) p.trace[g * 8 + 5] = clock64();
                    announce();
                    if (tr) p.trace[g * 8 + 6] = clock64();
                    if (g >= S) ok = mbar_wait(&empty[s], ((g / S) - 1) & 1, abort_flag);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after_sync();
                    if (tr) p.trace[g * 8 + 7] = clock64();
                    tmem_st_32x32b_x32(lane_base + (uint32_t)(D_COLS + s * A_COLS + a * 32), vals);
                    pending = s;
                    if (PH == 1) announce();          // a lone warp per weight rows: nothing to overlap the store with
                }
            }
        }
        if (ok) announce();
        else *abort_flag = 1;
    } else if (warp < NEXP + NEPI) {
        // ================= epilogue: TMEM -> registers -> global
        const int e = warp - NEXP;
        const int quarter = e & 3;                                        // == warp & 3: the lanes this warp may read
        constexpr int GROUPS = NEPI / 4;                                  // warps per lane quarter: they split the token columns
        const int grp = e >> 2;
        const uint32_t lane_base = tmem_base + ((uint32_t)(quarter * 32) << 16);
        constexpr int NCH = BN / 32;                                      // 32-column chunks of the tile
        constexpr int CH = (NCH + GROUPS - 1) / GROUPS;                   // chunks per warp
        constexpr int NOUT = (EPI == kEpiSiluMul) ? 1 : NA;               // output tiles per weight row
        constexpr bool HOLD = (NOUT * CH <= 6);                           // few chunks: read all, release, then store
        pdl_wait();                                                       // the output buffer may be in use upstream
        bool ok = true;
        int it = 0;
        // one 32-column chunk of output tile o: accumulators -> fp16 pairs (two tokens per register)
        auto read_chunk = [&](int o, int c0, uint32_t (&dst)[16]) {
            uint32_t v[32];
            tmem_ld_32x32b_x32(lane_base + (uint32_t)(o * BN + c0), v);
            if (EPI == kEpiSiluMul) {
                uint32_t u[32];
                tmem_ld_32x32b_x32(lane_base + (uint32_t)(BN + c0), u);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(silu_f(__uint_as_float(v[j])) * __uint_as_float(u[j]));
            } else {
                tmem_wait_ld();
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) dst[j] = as_u32(__floats2half2_rn(__uint_as_float(v[2 * j]), __uint_as_float(v[2 * j + 1])));
        };
        auto store_chunk = [&](int o, int c0, int row0, int rows, int n, const uint32_t (&src)[16]) {
            uint16_t* out = p.out + (size_t)(row0 + c0) * p.ldo + (size_t)o * p.a_col_offset + n;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                if (c0 + 2 * j < rows) out[(size_t)(2 * j) * p.ldo] = (uint16_t)(src[j] & 0xFFFFu);
                if (c0 + 2 * j + 1 < rows) out[(size_t)(2 * j + 1) * p.ldo] = (uint16_t)(src[j] >> 16);
            }
        };
        auto release = [&]() {                                            // the next tile may overwrite the accumulators
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty);
        };
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
            int n_tile, expert, row0, rows, ks;
            tile_rows(t, n_tile, expert, row0, rows, ks);
            ok = mbar_wait(acc_full, it & 1, abort_flag);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after_sync();
            const int n = n_tile * 128 + quarter * 32 + lane;             // weight row within the tile set
            if (splits > 1) {
                // split-K: fp32 partial sums of this split, [split][token][weight row]; a second kernel adds the splits
                if constexpr (EPI == kEpiStore) {
                    float* pbase = p.partial + ((size_t)ks * p.M + row0) * p.ldo + n;
#pragma unroll
                    for (int o = 0; o < NOUT; ++o) {
#pragma unroll
                        for (int c = 0; c < CH; ++c) {
                            const int c0 = (grp * CH + c) * 32;
                            if (c0 < BN && c0 < rows) {
                                uint32_t v[32];
                                tmem_ld_32x32b_x32(lane_base + (uint32_t)(o * BN + c0), v);
                                tmem_wait_ld();
                                float* dst = pbase + (size_t)c0 * p.ldo + (size_t)o * p.a_col_offset;
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    if (c0 + j < rows) dst[(size_t)j * p.ldo] = __uint_as_float(v[j]);
                            }
                        }
                    }
                }
                release();
            } else if constexpr (HOLD) {
                uint32_t packed[NOUT][CH][16];
#pragma unroll
                for (int o = 0; o < NOUT; ++o) {
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const int c0 = (grp * CH + c) * 32;
                        if (c0 < BN && c0 < rows) read_chunk(o, c0, packed[o][c]);   // uniform over the warp
                    }
                }
                release();
#pragma unroll
                for (int o = 0; o < NOUT; ++o) {
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const int c0 = (grp * CH + c) * 32;
                        if (c0 < BN && c0 < rows) store_chunk(o, c0, row0, rows, n, packed[o][c]);
                    }
                }
            } else {
                // many chunks: stream them (read, store), release after the last read
                uint32_t buf[16];
                bool pending = false;
                int po = 0, pc0 = 0;
#pragma unroll
                for (int o = 0; o < NOUT; ++o) {
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const int c0 = (grp * CH + c) * 32;
                        if (c0 < BN && c0 < rows) {
                            if (pending) store_chunk(po, pc0, row0, rows, n, buf);
                            read_chunk(o, c0, buf);
                            pending = true;
                            po = o;
                            pc0 = c0;
                        }
                    }
                }
                release();
                if (pending) store_chunk(po, pc0, row0, rows, n, buf);
            }
        }
        if (!ok) *abort_flag = 1;
    } else if (warp == TMA_WARP) {
        // ================= TMA producer: activation tiles
        if (lane == 0) {
            pdl_wait();                                                   // activations come from the previous kernel
            int issued = 0, g = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                int n_tile, expert, row0, rows, ks;
                tile_rows(t, n_tile, expert, row0, rows, ks);
                for (int kb = 0; kb < num_kb; ++kb, ++g) {
                    const int s = g % S;
                    if (g >= S) ok = mbar_wait(&empty[s], ((g / S) - 1) & 1, abort_flag);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&full[s], B_STAGE);
                    tma_load_2d(smem_b + s * B_STAGE, &x_map, (ks * num_kb + kb) * kGemmBK, row0, &full[s]);
                    issued = g + 1;
                }
            }
            if (!ok) {
                *abort_flag = 1;
                // let loads in flight land before the block's shared memory is released
                // (the same barrier also counts expander arrivals, so this can run into its time limit)
                for (int q = max(0, issued - S); q < issued; ++q) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&full[q % S], (q / S) & 1) && clock64() - t0 < (1LL << 22)) {}
                }
            }
        }
    } else {
        // ================= MMA issuer
        // The whole warp runs the loop converged (so that addresses and descriptors stay warp-uniform
        // values); one elected lane issues the MMAs and the commits.
        constexpr uint32_t idesc = idesc_f16_m128(BN);
        const uint64_t desc0 = smem_desc_k_sw128(smem_u32(smem_b));       // slot 0, k-step 0
        bool ok = true;
        int g = 0, it = 0;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, ++it) {
            if (it > 0) {                                                 // the epilogue must have read the accumulators
                ok = mbar_wait(acc_empty, (it - 1) & 1, abort_flag);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after_sync();
            }
            for (int kb = 0; kb < num_kb; ++kb, ++g) {
                const int s = g % S;
                const bool tr = p.trace != nullptr && blockIdx.x == 0 && g < 64 && lane == 0;
                if (tr) p.trace[g * 8 + 0] = clock64();
                ok = mbar_wait(&full[s], (g / S) & 1, abort_flag);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (tr) p.trace[g * 8 + 2] = clock64();
                if (!ok) break;
                tc_fence_after_sync();
                // descriptor start address is in 16-byte units: slot s is s * B_STAGE / 16 further, k-step k is 2 further
                const uint64_t desc_s = desc0 + (uint64_t)(s * (B_STAGE >> 4));
                const uint32_t a_s = tmem_base + (uint32_t)(D_COLS + s * A_COLS);
                if (elect_one()) {
#pragma unroll
                    for (int a = 0; a < NA; ++a) {
#pragma unroll
                        for (int k = 0; k < kGemmBK / 16; ++k)
                            mma_ts_f16(tmem_base + (uint32_t)(a * BN), a_s + (uint32_t)(a * 32 + k * 8), desc_s + (uint64_t)(k * 2), idesc,
                                       (kb | k) != 0);
                    }
                    mma_commit(&empty[s]);                                // slot reusable when these MMAs finish
                }
                __syncwarp();
                if (tr) p.trace[g * 8 + 3] = clock64();
            }
            if (ok && elect_one()) mma_commit(acc_full);                  // accumulators of this tile are complete
            __syncwarp();
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
