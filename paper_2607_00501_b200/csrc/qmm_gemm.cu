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

// The workspace of qmm_gemm holds only the device status word.
size_t gemm_workspace_bytes(int, int64_t, int64_t, int64_t) { return 256; }

qmm_status launch_gemm(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* X, int64_t ldx,
                       uint16_t* Y, int64_t ldy, int64_t M, void* ws, cudaStream_t st)
{
    // Token tile: 256 (the widest MMA, N = 256) once M exceeds one 128-token tile; one weight tile
    // per block, so that small problems spread over as many SMs as possible.
    int bn = M > 128 ? 256 : pick_token_tile(M);
    int na = 1;
    if (const char* f = getenv("QMM_GEMM_FORCE")) {            // "bn,na" for tuning sweeps
        int b = 0, a = 0;
        if (sscanf(f, "%d,%d", &b, &a) == 2 && (a == 1 || (a == 2 && N % 256 == 0 && b <= 128)) &&
            (b == 32 || b == 64 || b == 128 || (b == 256 && a == 1))) {
            bn = b;
            na = a;
        }
    }
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
    p.status = (int*)ws;
    if (getenv("QMM_GEMM_TRACE")) p.trace = (long long*)((uint8_t*)ws + 256);   // tuning aid: needs a workspace of >= 256 + 4096 bytes
    const int64_t tiles = (N / (128 * na)) * ((M + bn - 1) / bn);
    return launch_tc_gemm(fmt, bn, na, kEpiStore, map, p, persistent_grid(bn, na, tiles), st);
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
