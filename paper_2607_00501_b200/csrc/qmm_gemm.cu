// qmm_gemm.cu -- host side of the tensor-core products: TMA descriptors, tile
// selection and launches for the dense prefill GEMM (qmm_gemm) and, through
// launch_tc_gemm, the grouped expert GEMMs of qmm_moe.
#include "qmm_gemm_kernel.cuh"

#include <math.h>
#include <stdio.h>
#include <stdlib.h>

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

template <int FMT, int BN, int NA, int EPI>
static qmm_status launch_t(const CUtensorMap& map, const GemmParams& p, dim3 grid, cudaStream_t st)
{
    auto kern = gemm_kernel<FMT, BN, NA, EPI>;
    constexpr int smem = GemmGeom<BN, NA>::kSmemBytes;
    static bool configured = false;                 // per instantiation; attribute is sticky per device context
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return check_cuda(e, "tensor-core GEMM shared memory size");
        configured = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(GemmGeom<BN, NA>::kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return check_cuda(cudaLaunchKernelEx(&cfg, kern, map, p), "tensor-core GEMM launch");
}

// Launch one tensor-core product.  bn in {32, 64, 128}; na in {1, 2}; epi as GemmEpilogue.
qmm_status launch_tc_gemm(int fmt, int bn, int na, int epi, const CUtensorMap& map, const GemmParams& p, dim3 grid,
                          cudaStream_t st)
{
#define QMM_TC_CASE(F, B, A, E) \
    if (fmt == F && bn == B && na == A && epi == E) return launch_t<F, B, A, E>(map, p, grid, st);
#define QMM_TC_FMT(F)                     \
    QMM_TC_CASE(F, 32, 1, kEpiStore)      \
    QMM_TC_CASE(F, 64, 1, kEpiStore)      \
    QMM_TC_CASE(F, 128, 1, kEpiStore)     \
    QMM_TC_CASE(F, 256, 1, kEpiStore)     \
    QMM_TC_CASE(F, 32, 2, kEpiStore)      \
    QMM_TC_CASE(F, 64, 2, kEpiStore)      \
    QMM_TC_CASE(F, 128, 2, kEpiStore)     \
    QMM_TC_CASE(F, 160, 2, kEpiStore)     \
    QMM_TC_CASE(F, 32, 2, kEpiSiluMul)    \
    QMM_TC_CASE(F, 64, 2, kEpiSiluMul)    \
    QMM_TC_CASE(F, 128, 2, kEpiSiluMul)   \
    QMM_TC_CASE(F, 160, 2, kEpiSiluMul)
    QMM_TC_FMT(QMM_Q4)
    QMM_TC_FMT(QMM_Q8)
#undef QMM_TC_FMT
#undef QMM_TC_CASE
    return fail(QMM_ERR_UNSUPPORTED, "no tensor-core kernel for fmt=%d bn=%d na=%d epi=%d", fmt, bn, na, epi);
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

// Second stage of the split-K GEMM: Y[m][n] = fp16(sum_s partial[s][m][n]), s ascending (fixed order).
__global__ void gemm_splitk_reduce_kernel(const float* __restrict__ partial, uint16_t* __restrict__ Y, int M, int N,
                                          int64_t ldy, int splits)
{
    pdl_launch_dependents();
    pdl_wait();
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;      // one thread: 8 consecutive n of one m
    const int per_row = N / 8;
    if (i >= (int64_t)M * per_row) return;
    const int m = (int)(i / per_row), n = (int)(i % per_row) * 8;
    float acc[8];
    const float4* src = reinterpret_cast<const float4*>(partial + (size_t)m * N + n);
    float4 a = src[0], b = src[1];
    acc[0] = a.x; acc[1] = a.y; acc[2] = a.z; acc[3] = a.w;
    acc[4] = b.x; acc[5] = b.y; acc[6] = b.z; acc[7] = b.w;
    for (int s = 1; s < splits; ++s) {
        src = reinterpret_cast<const float4*>(partial + ((size_t)s * M + m) * N + n);
        a = src[0];
        b = src[1];
        acc[0] += a.x; acc[1] += a.y; acc[2] += a.z; acc[3] += a.w;
        acc[4] += b.x; acc[5] += b.y; acc[6] += b.z; acc[7] += b.w;
    }
    uint4 o;
    __half2* oh = reinterpret_cast<__half2*>(&o);
#pragma unroll
    for (int j = 0; j < 4; ++j) oh[j] = __floats2half2_rn(acc[2 * j], acc[2 * j + 1]);
    uint16_t* dst = Y + (size_t)m * ldy + n;
    if ((reinterpret_cast<uintptr_t>(dst) & 15) == 0) {
        *reinterpret_cast<uint4*>(dst) = o;
    } else {                                                              // a row pitch that is not a multiple of 8
        const uint16_t* oh16 = reinterpret_cast<const uint16_t*>(&o);
#pragma unroll
        for (int j = 0; j < 8; ++j) dst[j] = oh16[j];
    }
}

// Shape -> tiling of the dense GEMM.
struct GemmPlan {
    int bn, na, splits;
};

// Token tile: 256 (the widest MMA, N = 256) once M exceeds one 128-token tile; one weight tile per
// block.  When the tiles cannot cover the SMs, the K range is split across blocks (fp32 partial
// sums in the workspace, a second stage adds them in a fixed order), as long as every split keeps
// at least 8 k-blocks and an even number of them.
static GemmPlan gemm_plan(int64_t M, int64_t N, int64_t K)
{
    GemmPlan p;
    p.bn = M > 128 ? 256 : pick_token_tile(M);
    p.na = 1;
    p.splits = 1;
    const int64_t tiles = (N / 128) * ((M + p.bn - 1) / p.bn);
    const int num_kb = (int)(K / kGemmBK);
    while (tiles * p.splits * 2 <= kNumSMs && num_kb % (p.splits * 2) == 0 && num_kb / (p.splits * 2) >= 8 &&
           (num_kb / (p.splits * 2)) % 2 == 0)
        p.splits *= 2;
    if (const char* f = getenv("QMM_GEMM_FORCE")) {            // "bn,na[,splits]" for tuning sweeps and tests
        int b = 0, a = 0, sp = 1;
        const int got = sscanf(f, "%d,%d,%d", &b, &a, &sp);
        if (got >= 2 && (a == 1 || (a == 2 && N % 256 == 0 && b <= 128)) &&
            (b == 32 || b == 64 || b == 128 || (b == 256 && a == 1))) {
            p.bn = b;
            p.na = a;
            p.splits = 1;
            if (got == 3 && sp >= 1 && num_kb % sp == 0 && (num_kb / sp) % 2 == 0) p.splits = sp;
        }
    }
    return p;
}

// Workspace of qmm_gemm: the device status word, then the split-K partial sums.
size_t gemm_workspace_bytes(int, int64_t M, int64_t N, int64_t K)
{
    const GemmPlan p = gemm_plan(M, N, K);
    return 256 + (p.splits > 1 ? (size_t)p.splits * (size_t)M * (size_t)N * sizeof(float) : 0);
}

qmm_status launch_gemm(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* X, int64_t ldx,
                       uint16_t* Y, int64_t ldy, int64_t M, void* ws, cudaStream_t st)
{
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
    p.ldo = plan.splits > 1 ? N : ldy;                                    // partial sums are [split][M][N], dense
    p.a_col_offset = (int)(N / 2);
    p.M = (int)M;
    p.splits = plan.splits;
    p.partial = plan.splits > 1 ? (float*)((uint8_t*)ws + 256) : nullptr;
    p.status = (int*)ws;
    if (getenv("QMM_GEMM_TRACE") && plan.splits == 1)
        p.trace = (long long*)((uint8_t*)ws + 256);                       // tuning aid: needs a workspace of >= 256 + 4096 bytes
    const int64_t tiles = (N / (128 * na)) * ((M + bn - 1) / bn) * plan.splits;
    s = launch_tc_gemm(fmt, bn, na, kEpiStore, map, p, persistent_grid(bn, na, tiles), st);
    if (s != QMM_OK || plan.splits == 1) return s;
    cudaLaunchConfig_t cfg = {};
    const int64_t threads = M * (N / 8);
    cfg.gridDim = dim3((unsigned)((threads + 255) / 256));
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return check_cuda(cudaLaunchKernelEx(&cfg, gemm_splitk_reduce_kernel, (const float*)p.partial, Y, (int)M, (int)N,
                                         (int64_t)ldy, plan.splits),
                      "qmm_gemm split-K reduce launch");
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
        return fail(QMM_ERR_CUDA, "device status word holds unexpected value %d", h);
    }
    return QMM_OK;
}

}  // namespace qmm
