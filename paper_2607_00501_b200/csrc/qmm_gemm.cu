// qmm_gemm.cu -- host side of the tensor-core products: TMA descriptors, tile
// selection and launches for the dense prefill GEMM (qmm_gemm) and, through
// launch_tc_gemm, the grouped expert GEMMs of qmm_moe.
#include "qmm_gemm_kernel.cuh"

#include <atomic>
#include <math.h>
#include <stdio.h>

namespace qmm {

// cuTensorMapEncodeTiled is reached through the runtime so that libqmm links
// against the CUDA runtime only.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// fp16 [rows, ld] row-major, tiles of 64 k x box_rows rows, 128-byte swizzle,
// out-of-range rows read as zero.
qmm_status make_x_map(CUtensorMap* map, const uint16_t* X, int64_t rows, int64_t K, int64_t ld, int box_rows)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(QMM_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    const cuuint64_t gdim[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kGemmBK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<uint16_t*>(X), gdim, gstride, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(QMM_ERR_CUDA, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return QMM_OK;
}

template <int FMT, int BN, int NA, int EPI, bool DENSE>
static qmm_status launch_t(const CUtensorMap& map, const GemmParams& p, dim3 grid, cudaStream_t st)
{
    auto kern = gemm_kernel<FMT, BN, NA, EPI, DENSE>;
    constexpr int smem = GemmGeom<BN, NA, EPI, FMT>::kSmemBytes;
    // the attribute is per device: remember which devices have it (per instantiation)
    static std::atomic<uint64_t> configured{0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) dev = 0;
    const uint64_t bit = dev < 64 ? (1ull << dev) : 0;
    if (!(configured.load(std::memory_order_relaxed) & bit)) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return check_cuda(e, "tensor-core GEMM shared memory size");
        configured.fetch_or(bit, std::memory_order_relaxed);
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(GemmGeom<BN, NA, EPI, FMT>::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return check_cuda(cudaLaunchKernelEx(&cfg, kern, map, p), "tensor-core GEMM launch");
}

// Launch one tensor-core product.  Dense (qmm_gemm): one weight tile set, token tiles of 32 .. 256,
// plain store.  Grouped (expert products): token tiles of 32 .. 160 from a device-built list, one
// or two weight tile sets, plain store or SiLU*mul.
qmm_status launch_tc_gemm(int fmt, int bn, int na, int epi, bool dense, const CUtensorMap& map, const GemmParams& p,
                          dim3 grid, cudaStream_t st)
{
#define QMM_TC_CASE(F, B, A, E, D) \
    if (fmt == F && bn == B && na == A && epi == E && dense == D) return launch_t<F, B, A, E, D>(map, p, grid, st);
#define QMM_TC_FMT(F)                            \
    QMM_TC_CASE(F, 32, 1, kEpiStore, true)       \
    QMM_TC_CASE(F, 64, 1, kEpiStore, true)       \
    QMM_TC_CASE(F, 128, 1, kEpiStore, true)      \
    QMM_TC_CASE(F, 160, 1, kEpiStore, true)      \
    QMM_TC_CASE(F, 192, 1, kEpiStore, true)      \
    QMM_TC_CASE(F, 256, 1, kEpiStore, true)      \
    QMM_TC_CASE(F, 32, 1, kEpiStore, false)      \
    QMM_TC_CASE(F, 64, 1, kEpiStore, false)      \
    QMM_TC_CASE(F, 128, 1, kEpiStore, false)     \
    QMM_TC_CASE(F, 160, 1, kEpiStore, false)     \
    QMM_TC_CASE(F, 32, 2, kEpiStore, false)      \
    QMM_TC_CASE(F, 64, 2, kEpiStore, false)      \
    QMM_TC_CASE(F, 128, 2, kEpiStore, false)     \
    QMM_TC_CASE(F, 160, 2, kEpiStore, false)     \
    QMM_TC_CASE(F, 32, 2, kEpiSiluMul, false)    \
    QMM_TC_CASE(F, 64, 2, kEpiSiluMul, false)    \
    QMM_TC_CASE(F, 128, 2, kEpiSiluMul, false)   \
    QMM_TC_CASE(F, 160, 2, kEpiSiluMul, false)
    QMM_TC_FMT(QMM_Q4)
    QMM_TC_FMT(QMM_Q8)
#undef QMM_TC_FMT
#define QMM_TC_DENSE_ONLY(F)                     \
    QMM_TC_CASE(F, 32, 1, kEpiStore, true)       \
    QMM_TC_CASE(F, 64, 1, kEpiStore, true)       \
    QMM_TC_CASE(F, 128, 1, kEpiStore, true)      \
    QMM_TC_CASE(F, 160, 1, kEpiStore, true)      \
    QMM_TC_CASE(F, 192, 1, kEpiStore, true)      \
    QMM_TC_CASE(F, 256, 1, kEpiStore, true)
    QMM_TC_DENSE_ONLY(QMM_Q5)                     // the 5- and 6-bit formats: dense product only
    QMM_TC_DENSE_ONLY(QMM_Q6)
#undef QMM_TC_DENSE_ONLY
#undef QMM_TC_CASE
    return fail(QMM_ERR_UNSUPPORTED, "no tensor-core kernel for fmt=%d bn=%d na=%d epi=%d dense=%d", fmt, bn, na, epi, (int)dense);
}

// Persistent grid: one block per SM (a block's 18 warps use most of the register file), never
// more blocks than tiles (tiles <= 0: unknown on the host, the kernel reads the count).
dim3 persistent_grid(int bn, int na, int64_t tiles)
{
    (void)bn;
    (void)na;
    int64_t g = kNumSMs;
    if (tiles > 0 && tiles < g) g = tiles;
    return dim3((unsigned)g);
}

int pick_token_tile(int64_t rows)
{
    return rows <= 32 ? 32 : rows <= 64 ? 64 : 128;
}

// Token tile of the grouped (per-expert) GEMMs: the smallest tile that holds the mean number of rows
// per expert plus three standard deviations of a uniform routing (binomial), so that almost every
// expert is one tile.  160 is the widest two-accumulator tile that leaves tensor memory for a 3-slot ring.
int pick_expert_tile(int64_t total_rows, int experts)
{
    const double mean = (double)total_rows / experts;
    const double want = mean + 3.0 * sqrt(mean) + 1.0;
    return want <= 32 ? 32 : want <= 64 ? 64 : want <= 128 ? 128 : 160;
}

// Adds the partial sums of the tiles that the dense GEMM cut across blocks, contributors in
// ascending order (a fixed order: same bits on every call), and stores fp16.  Block (t, y): token columns [8 y, 8 y + 8) of tile t; a
// thread adds one float4 (4 weight rows of one token) per output tile, so every load is in flight at once.
__global__ void gemm_cut_reduce_kernel(const float* __restrict__ partial, uint16_t* __restrict__ Y, int64_t ldy, int M,
                                       int bn, int nout, int a_col_offset, int n_tiles, int KB, int U, int t0)
{
    pdl_launch_dependents();
    pdl_wait();
    const int t = t0 + blockIdx.x, c0 = blockIdx.y * 8;                   // the tiles dealt in unit shares start at t0
    const int n_tile = t % n_tiles, row0 = (t / n_tiles) * bn;
    const int rows = min(bn, M - row0);
    if (c0 >= rows) return;
    const long long tb = (long long)blockIdx.x * KB;
    const int first = (int)(tb / U);
    const int cn = (int)((tb + KB - 1) / U) - first + 1;
    if (cn == 1) return;                                                  // a whole tile: stored by the GEMM itself
    const size_t slot = (size_t)nout * bn * 128;
    const int r4 = threadIdx.x & 31, j = threadIdx.x >> 5;                 // 4 weight rows, token column
    if (c0 + j >= rows) return;
    for (int o = 0; o < nout; ++o) {
        const size_t off = (size_t)(o * bn + c0 + j) * 128 + r4 * 4;
        float4 acc = __ldcg(reinterpret_cast<const float4*>(partial + (size_t)(2 * first + 1) * slot + off));
        for (int c = 1; c < cn; ++c) {
            const float4 v = __ldcg(reinterpret_cast<const float4*>(partial + (size_t)(2 * (first + c)) * slot + off));
            acc.x += v.x;
            acc.y += v.y;
            acc.z += v.z;
            acc.w += v.w;
        }
        uint2 h;
        *reinterpret_cast<__half2*>(&h.x) = __floats2half2_rn(acc.x, acc.y);
        *reinterpret_cast<__half2*>(&h.y) = __floats2half2_rn(acc.z, acc.w);
        *reinterpret_cast<uint2*>(Y + (size_t)(row0 + c0 + j) * ldy + (size_t)o * a_col_offset + n_tile * 128 + r4 * 4) = h;
    }
}

// Shape -> tiling and work split of the dense GEMM.
struct GemmPlan {
    int bn, na;
    int whole;          // tiles dealt whole, the same number to every block (a multiple of grid)
    bool halves;        // the remaining tiles are dealt as half tiles (BN / 2 tokens each)
    int units;          // (tile, k-block) units per block of the remaining tiles
    int grid;           // blocks
    bool cut;           // some tile is shared between blocks: partial-sum slots and the second kernel
};

// Cycles of one block for `tiles` tiles of `kb` k-blocks on the SMs: whole rounds, then the last,
// partly filled round either as whole tiles or -- when that saves more than the partial sums and
// the second kernel cost (~18 000 cycles, measured) -- cut into equal shares of its (tile, k-block) units.
struct RoundCost {
    int64_t cycles;
    bool cut_tail;
    bool halve_tail;    // instead: the last round's tiles as two half tiles each (256-token tiles, at most SMs / 2 of them)
};
static RoundCost round_cost(int64_t tiles, int64_t kb, int64_t stage, int64_t handover)
{
    const int64_t tile = kb * stage + handover;
    const int64_t rounds = tiles / kNumSMs, tail = tiles % kNumSMs;
    RoundCost r = {rounds * tile, false, false};
    if (tail == 0) return r;
    int64_t share = (tail * kb + kNumSMs - 1) / kNumSMs;
    if (share < 8) share = 8;
    const int64_t cut = share * stage + 2 * handover + 18000;
    // half tiles (N = 128 MMAs in the 256-token kernel): ~470 cycles per stage, measured
    const int64_t halves = (stage == 515 && 2 * tail <= kNumSMs) ? kb * 470 + handover : tile + 1;
    if (rounds >= 1 && halves < tile && halves <= cut) {
        r.cycles += halves;
        r.halve_tail = true;
    } else if (rounds >= 1 && cut < tile) {
        r.cycles += cut;
        r.cut_tail = true;
    } else {
        r.cycles += tile;
    }
    return r;
}

// Workspace of qmm_gemm: [0, 4) status word, [4096, 8192) trace samples (tuning aid), then the
// partial-sum slots.
[[maybe_unused]] constexpr size_t kGemmWsTrace = 4096;
constexpr size_t kGemmWsHeader = 8192;

// Token tile: 256 (the widest MMA, N = 256) once M exceeds one 128-token tile, else the smallest
// that holds M -- or half / a quarter of that when this yields between 3/4 and one round of whole
// tiles; one weight tile per block.  Work split:
//   tiles <= SMs / 2: every tile is cut into equal pieces along K, one per block, as many as the
//                     SMs can take at once; a second kernel adds the pieces;
//   otherwise:        whole tiles, the same number for every block, and for the tiles of the
//                     last, partly filled round the cheapest of (round_cost): whole tiles on
//                     some of the SMs; equal shares of their (tile, k-block) units on all SMs
//                     (partial sums + second kernel); two half tiles each (256-token tiles, at
//                     most SMs / 2 of them left).  Cutting *every* tile into shares was measured
//                     too: the fp32 partial traffic costs more than it saves.
static GemmPlan gemm_plan(int64_t M, int64_t N, int64_t K)
{
    GemmPlan p;
    p.bn = M > 128 ? 256 : pick_token_tile(M);
    p.na = 1;
    // a narrower token tile that fills one round of the SMs with whole tiles beats cutting K
    // (no partial sums, no second kernel)
    for (int cand = p.bn / 2; cand >= 64 && (N / 128) * ((M + p.bn - 1) / p.bn) * 2 <= kNumSMs; cand /= 2) {
        const int64_t t = (N / 128) * ((M + cand - 1) / cand);
        if (t * 4 >= (int64_t)kNumSMs * 3 && t <= kNumSMs) {
            p.bn = cand;
            break;
        }
    }
    // many tiles: 256 tokens (N = 256 MMAs at the tensor rate, but one accumulator buffer: ~2 400 cycles
    // of hand-over per tile) or 192 (two accumulator buffers, ~470 cycles per stage against 515):
    // whichever needs fewer cycles for its rounds of whole tiles on the SMs
    if (p.bn == 256 && (N / 128) * ((M + 255) / 256) * 2 > kNumSMs) {
        const int64_t kb = K / kGemmBK;
        const int64_t t256 = (N / 128) * ((M + 255) / 256), t192 = (N / 128) * ((M + 191) / 192);
        if (round_cost(t192, kb, 470, 300).cycles < round_cost(t256, kb, 515, 2400).cycles) p.bn = 192;
    }
    int force_units = 0;
    if (g_knobs.gemm_bn) {                                      // forced by qmm_debug_config("gemm_force", "bn[,units]")
        p.bn = g_knobs.gemm_bn;
        force_units = g_knobs.gemm_units;
    }
    const int64_t tiles = (N / (128 * p.na)) * ((M + p.bn - 1) / p.bn);
    const int64_t KB = K / kGemmBK;
    const int64_t total = tiles * KB;
    int64_t units;
    p.whole = 0;
    p.grid = 0;
    p.halves = false;
    if (tiles * 2 > kNumSMs && !force_units) {
        // whole tiles, the same number for every block; the tiles of the last, partly filled round
        // are cut into equal shares of their units when round_cost says that pays
        const RoundCost rc = p.bn == 256 ? round_cost(tiles, KB, 515, 2400) : round_cost(tiles, KB, 470, 300);
        if (rc.halve_tail && !g_knobs.gemm_no_tail_cut) {
            p.grid = kNumSMs;
            p.whole = (int)(tiles / kNumSMs) * kNumSMs;
            p.halves = true;
            p.units = (int)KB;
            p.cut = false;
            return p;
        }
        if (rc.cut_tail && !g_knobs.gemm_no_tail_cut) {
            p.grid = kNumSMs;
            p.whole = (int)(tiles / kNumSMs) * kNumSMs;
            units = ((tiles - p.whole) * KB + kNumSMs - 1) / kNumSMs;
            if (units < 8) units = 8;
            p.units = (int)units;
            p.cut = true;
            return p;
        }
    }
    if (tiles * 2 <= kNumSMs) {
        // the largest number of equal pieces per tile that the SMs can take at once, every piece
        // worth a pipeline fill and an epilogue (>= 8 k-blocks)
        int64_t pieces = 1;
        for (int64_t d = 2; d * tiles <= kNumSMs; ++d)
            if (KB % d == 0 && KB / d >= 8) pieces = d;
        units = KB / pieces;
    } else {
        units = KB * ((tiles + kNumSMs - 1) / kNumSMs);       // whole tiles, the same number for every block
    }
    if (force_units) units = force_units;
    p.units = (int)units;
    p.grid = (int)((total + units - 1) / units);
    p.cut = units % KB != 0;
    return p;
}

// defined in qmm_gemm_small.cu
bool gemm_small_supported(int fmt, int64_t M);
qmm_status launch_gemm_small(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* X, int64_t ldx,
                             uint16_t* Y, int64_t ldy, int64_t M, cudaStream_t st);

size_t gemm_workspace_bytes(int, int64_t M, int64_t N, int64_t K)
{
    if (M == 0) return kGemmWsHeader;
    const GemmPlan p = gemm_plan(M, N, K);
    return kGemmWsHeader + (p.cut ? (size_t)2 * p.grid * p.na * p.bn * 128 * sizeof(float) : 0);
}

qmm_status launch_gemm(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* X, int64_t ldx,
                       uint16_t* Y, int64_t ldy, int64_t M, void* ws, cudaStream_t st)
{
    // a handful of tokens: bound by streaming W once, like decode -- the few-token kernel
    if (gemm_small_supported(fmt, M)) return launch_gemm_small(fmt, packed, N, K, X, ldx, Y, ldy, M, st);
    const GemmPlan plan = gemm_plan(M, N, K);
    const int bn = plan.bn, na = plan.na;
    CUtensorMap map;
    qmm_status s = make_x_map(&map, X, M, K, ldx, bn);
    if (s != QMM_OK) return s;
    GemmParams p = {};
    const size_t half_bytes = (size_t)(N / 2 / kRowsPerGroup) * (size_t)(K / tile_k_of(fmt)) * tile_bytes_of(fmt);
    p.w[0] = (const uint8_t*)packed;
    p.w[1] = na == 2 ? (const uint8_t*)packed + half_bytes : nullptr;     // second tile set = lower half of the rows
    p.w_expert_stride = 0;
    p.N = (int)N;
    p.K = (int)K;
    p.out = Y;
    p.ldo = ldy;
    p.a_col_offset = (int)(N / 2);
    p.M = (int)M;
    p.whole_tiles = plan.whole;
    p.tail_halves = plan.halves ? 1 : 0;
    p.units_per_block = plan.units;
    p.partial = (float*)((uint8_t*)ws + kGemmWsHeader);
    p.status = (int*)ws;
#if QMM_GEMM_TRACE
    p.trace = (long long*)((uint8_t*)ws + kGemmWsTrace);                   // tuning builds only
#endif
    s = launch_tc_gemm(fmt, bn, na, kEpiStore, true, map, p, dim3((unsigned)plan.grid), st);
    if (s != QMM_OK || !plan.cut) return s;
    const int n_tiles = (int)(N / (128 * na));
    const int64_t tiles = (int64_t)n_tiles * ((M + bn - 1) / bn);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(tiles - plan.whole), (unsigned)(bn / 8));
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return check_cuda(cudaLaunchKernelEx(&cfg, gemm_cut_reduce_kernel, (const float*)p.partial, Y, (int64_t)ldy, (int)M, bn, na,
                                         p.a_col_offset, n_tiles, (int)(K / kGemmBK), plan.units, plan.whole),
                      "qmm_gemm partial-sum kernel launch");
}

// Debug aid: the give-up path of the bounded waits on its own.  One warp waits on an mbarrier that
// nobody ever arrives on, with a short limit; no TMA load and no tensor-core operation is in flight, so
// giving up has nothing to unwind.  The kernel then does what the GEMM kernels do on give-up: raise
// the abort flag, write QMM_ERR_DEVICE_TIMEOUT to the status word, return.
__global__ void wait_give_up_kernel(int* status, long long limit_cycles)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        abort_flag = 0;
        tc::fence_barrier_init();
    }
    __syncthreads();
    bool ok = tc::mbar_wait(&bar, 0, &abort_flag, limit_cycles);
    ok = __all_sync(0xFFFFFFFFu, ok);
    if (!ok) abort_flag = 1;
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) atomicExch(status, (int)QMM_ERR_DEVICE_TIMEOUT);
}

qmm_status launch_wait_give_up(int* status, long long limit_cycles, cudaStream_t st)
{
    wait_give_up_kernel<<<1, 32, 0, st>>>(status, limit_cycles);
    return check_cuda(cudaGetLastError(), "qmm_debug_wait_give_up launch");
}

// Reads and clears the device status word (first int of a GEMM / MoE workspace).
qmm_status status_check(void* ws, cudaStream_t st)
{
    int h = 0;
    cudaError_t e = cudaMemcpyAsync(&h, ws, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return check_cuda(e, "qmm_status_check");
    if (h != 0) {
        e = cudaMemsetAsync(ws, 0, sizeof(int), st);
        if (e == cudaSuccess) e = cudaStreamSynchronize(st);
        if (e != cudaSuccess) return check_cuda(e, "qmm_status_check");
        if (h == QMM_ERR_DEVICE_TIMEOUT)
            return fail(QMM_ERR_DEVICE_TIMEOUT, "a kernel gave up on a bounded wait (pipeline barrier never completed)");
        if (h == QMM_ERR_BAD_WEIGHTS)
            return fail(QMM_ERR_BAD_WEIGHTS, "qmm_packed_check found a scale that is inf/NaN or out of range: not a packed buffer of that format and shape");
        return fail(QMM_ERR_CUDA, "device status word holds unexpected value %d", h);
    }
    return QMM_OK;
}

}  // namespace qmm
