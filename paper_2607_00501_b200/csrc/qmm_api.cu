// qmm_api.cu -- the C ABI of libqmm: argument checks, error reporting, dispatch.
//
// Every entry point validates on the host, enqueues kernels on the caller's
// stream and returns; nothing here allocates device memory (the paper's
// runtime allocates nothing on its hot path and reports errors through a
// static thread-local buffer, Sec. 3.2 -- the same rules hold at this
// boundary).
#include "qmm_common.cuh"

#include <stdarg.h>
#include <stdio.h>
#include <string.h>

namespace qmm {

static thread_local char g_err[512] = "";

qmm_status fail(qmm_status code, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

qmm_status check_cuda(cudaError_t e, const char* what)
{
    if (e == cudaSuccess) return QMM_OK;
    return fail(QMM_ERR_CUDA, "%s: %s (%s)", what, cudaGetErrorString(e), cudaGetErrorName(e));
}

// defined in the kernel files
qmm_status launch_pack(int fmt, const void* canon, int64_t N, int64_t K, void* packed, cudaStream_t st);
qmm_status launch_dequant(int fmt, const void* packed, int64_t N, int64_t K, float* w_out, cudaStream_t st);
size_t gemv_workspace_bytes(int fmt, int64_t N, int64_t K, bool allow_cluster);
qmm_status launch_gemv(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* x, uint16_t* y,
                       void* ws, bool allow_cluster, cudaStream_t st);
qmm_status launch_gemv_batch(int fmt, const qmm_gemv_problem* probs, int count, cudaStream_t st, bool out_f32);
qmm_status launch_gemv_gate_up(int fmt, const void* packed_gate, const void* packed_up, int64_t N, int64_t K,
                               const uint16_t* x, uint16_t* h, cudaStream_t st);
size_t gemm_workspace_bytes(int fmt, int64_t M, int64_t N, int64_t K);
qmm_status launch_gemm(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* X, int64_t ldx,
                       uint16_t* Y, int64_t ldy, int64_t M, void* ws, cudaStream_t st);
qmm_status launch_gemm_small_batch(int fmt, const qmm_gemm_problem* probs, int count, int64_t M, cudaStream_t st);
size_t moe_workspace_bytes(const qmm_moe_args* a);
qmm_status launch_moe(const qmm_moe_args* a, void* ws, bool route_only, cudaStream_t st);
qmm_status status_check(void* ws, cudaStream_t st);
qmm_status launch_packed_check(int fmt, const void* packed, int64_t N, int64_t K, int* status, cudaStream_t st);
qmm_status launch_wait_give_up(int* status, long long limit_cycles, cudaStream_t st);

size_t chain_plan_bytes(int fmt, const qmm_chain_stage* st, int count);
size_t chain_workspace_bytes(int fmt, const qmm_chain_stage* st, int count);
qmm_status chain_build(int fmt, const qmm_chain_stage* st, int count, void* plan, size_t plan_bytes, void* ws, size_t ws_bytes,
                       qmm_chain_info* info, cudaStream_t stream);
qmm_status chain_run(const qmm_chain_info* info, cudaStream_t stream);

DebugKnobs g_knobs = {};

static bool fmt_ok(int fmt) { return fmt == QMM_Q4 || fmt == QMM_Q5 || fmt == QMM_Q6 || fmt == QMM_Q8; }

// Q5 and Q6 are built for pack / dequant / check, the single and the batched GEMV and the dense GEMM only.
static qmm_status check_fmt_everywhere(const char* who, int fmt)
{
    if (fmt == QMM_Q5 || fmt == QMM_Q6)
        return fail(QMM_ERR_UNSUPPORTED, "%s: format %d is built for qmm_pack, qmm_dequant, qmm_packed_check, qmm_gemv, qmm_gemv_batch, qmm_gemm and qmm_gemm_batch only", who, fmt);
    return QMM_OK;
}

static bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// The kernels are built for sm_100a only; refuse any other device.
static qmm_status check_device(const char* who)
{
    static thread_local int cached_dev = -1;
    static thread_local int cached_ok = 0;
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return check_cuda(e, who);
    if (dev != cached_dev) {
        int major = 0, minor = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e != cudaSuccess) return check_cuda(e, who);
        e = cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev);
        if (e != cudaSuccess) return check_cuda(e, who);
        cached_dev = dev;
        cached_ok = (major == 10 && minor == 0);
    }
    if (!cached_ok)
        return fail(QMM_ERR_UNSUPPORTED, "%s: device %d is not compute capability 10.0 (B200); no other target is built", who, dev);
    return QMM_OK;
}

// Shape rules shared by every call that takes a packed matrix.
static qmm_status check_matrix(const char* who, int fmt, int64_t N, int64_t K)
{
    if (!fmt_ok(fmt)) return fail(QMM_ERR_INVALID_ARG, "%s: unknown format %d (expected 4, 5, 6 or 8)", who, fmt);
    if (N <= 0 || K <= 0) return fail(QMM_ERR_INVALID_ARG, "%s: N=%lld and K=%lld must be positive", who, (long long)N, (long long)K);
    if (K % 32) return fail(QMM_ERR_SHAPE, "%s: K=%lld is not a multiple of the block size 32", who, (long long)K);
    if (K % 256) return fail(QMM_ERR_UNSUPPORTED, "%s: K=%lld is not a multiple of 256", who, (long long)K);
    if (N % 128) return fail(QMM_ERR_UNSUPPORTED, "%s: N=%lld is not a multiple of 128", who, (long long)N);
    if (N > (1 << 24) || K > (1 << 16))
        return fail(QMM_ERR_UNSUPPORTED, "%s: N=%lld > 2^24 or K=%lld > 2^16", who, (long long)N, (long long)K);
    return QMM_OK;
}

}  // namespace qmm

using namespace qmm;

extern "C" {

const char* qmm_last_error(void) { return g_err; }

int qmm_version(void) { return 100; }

size_t qmm_canonical_bytes(qmm_format fmt, int64_t N, int64_t K)
{
    if (!fmt_ok(fmt) || N <= 0 || K <= 0 || K % 32) return 0;
    return (size_t)N * (size_t)(K / 32) * (size_t)canon_block_of(fmt);
}

size_t qmm_packed_bytes(qmm_format fmt, int64_t N, int64_t K)
{
    if (check_matrix("qmm_packed_bytes", fmt, N, K) != QMM_OK) return 0;
    return (size_t)(N / kRowsPerGroup) * (size_t)(K / tile_k_of(fmt)) * (size_t)tile_bytes_of(fmt);
}

qmm_status qmm_pack(qmm_format fmt, const void* canonical, int64_t N, int64_t K, void* packed, void* stream)
{
    qmm_status s = check_matrix("qmm_pack", fmt, N, K);
    if (s != QMM_OK) return s;
    if (!canonical || !packed) return fail(QMM_ERR_INVALID_ARG, "qmm_pack: null pointer");
    if (!aligned(packed, 32)) return fail(QMM_ERR_ALIGNMENT, "qmm_pack: packed must be 32-byte aligned");
    if ((s = check_device("qmm_pack")) != QMM_OK) return s;
    return launch_pack(fmt, canonical, N, K, packed, (cudaStream_t)stream);
}

qmm_status qmm_dequant(qmm_format fmt, const void* packed, int64_t N, int64_t K, float* w_out, void* stream)
{
    qmm_status s = check_matrix("qmm_dequant", fmt, N, K);
    if (s != QMM_OK) return s;
    if (!packed || !w_out) return fail(QMM_ERR_INVALID_ARG, "qmm_dequant: null pointer");
    if (!aligned(packed, 32)) return fail(QMM_ERR_ALIGNMENT, "qmm_dequant: packed must be 32-byte aligned");
    if (!aligned(w_out, 16)) return fail(QMM_ERR_ALIGNMENT, "qmm_dequant: w_out must be 16-byte aligned");
    if ((s = check_device("qmm_dequant")) != QMM_OK) return s;
    return launch_dequant(fmt, packed, N, K, w_out, (cudaStream_t)stream);
}

size_t qmm_gemv_workspace_bytes(qmm_format fmt, int64_t N, int64_t K)
{
    if (check_matrix("qmm_gemv_workspace_bytes", fmt, N, K) != QMM_OK) return 0;
    return gemv_workspace_bytes(fmt, N, K, true);
}

qmm_status qmm_gemv(qmm_format fmt, const void* packed, int64_t N, int64_t K,
                    const uint16_t* x_fp16, uint16_t* y_fp16, void* ws, size_t ws_bytes, void* stream)
{
    qmm_status s = check_matrix("qmm_gemv", fmt, N, K);
    if (s != QMM_OK) return s;
    if (!packed || !x_fp16 || !y_fp16) return fail(QMM_ERR_INVALID_ARG, "qmm_gemv: null pointer");
    if (!aligned(packed, 32)) return fail(QMM_ERR_ALIGNMENT, "qmm_gemv: packed must be 32-byte aligned");
    if (!aligned(x_fp16, 16) || !aligned(y_fp16, 16))
        return fail(QMM_ERR_ALIGNMENT, "qmm_gemv: x and y must be 16-byte aligned");
    if (K > 32768) return fail(QMM_ERR_UNSUPPORTED, "qmm_gemv: K=%lld > 32768", (long long)K);
    const size_t need = gemv_workspace_bytes(fmt, N, K, true);
    if (need > 0) {
        if (!ws || ws_bytes < need)
            return fail(QMM_ERR_WORKSPACE, "qmm_gemv: workspace of %zu bytes needed, %zu given", need, ws ? ws_bytes : (size_t)0);
        if (!aligned(ws, 16)) return fail(QMM_ERR_ALIGNMENT, "qmm_gemv: workspace must be 16-byte aligned");
    }
    if ((s = check_device("qmm_gemv")) != QMM_OK) return s;
    return launch_gemv(fmt, packed, N, K, x_fp16, y_fp16, ws, true, (cudaStream_t)stream);
}

qmm_status qmm_gemv_gate_up(qmm_format fmt, const void* packed_gate, const void* packed_up, int64_t N, int64_t K,
                            const uint16_t* x_fp16, uint16_t* h_fp16, void* stream)
{
    qmm_status s = check_matrix("qmm_gemv_gate_up", fmt, N, K);
    if (s != QMM_OK) return s;
    if ((s = check_fmt_everywhere("qmm_gemv_gate_up", fmt)) != QMM_OK) return s;
    if (!packed_gate || !packed_up || !x_fp16 || !h_fp16) return fail(QMM_ERR_INVALID_ARG, "qmm_gemv_gate_up: null pointer");
    if (!aligned(packed_gate, 32) || !aligned(packed_up, 32))
        return fail(QMM_ERR_ALIGNMENT, "qmm_gemv_gate_up: packed matrices must be 32-byte aligned");
    if (!aligned(x_fp16, 16) || !aligned(h_fp16, 16))
        return fail(QMM_ERR_ALIGNMENT, "qmm_gemv_gate_up: x and h must be 16-byte aligned");
    if (K > 32768) return fail(QMM_ERR_UNSUPPORTED, "qmm_gemv_gate_up: K=%lld > 32768", (long long)K);
    if ((s = check_device("qmm_gemv_gate_up")) != QMM_OK) return s;
    return launch_gemv_gate_up(fmt, packed_gate, packed_up, N, K, x_fp16, h_fp16, (cudaStream_t)stream);
}

qmm_status qmm_gemv_batch(qmm_format fmt, const qmm_gemv_problem* problems, int count, void* stream)
{
    if (count < 0) return fail(QMM_ERR_INVALID_ARG, "qmm_gemv_batch: count=%d is negative", count);
    if (count == 0) return QMM_OK;
    if (!problems) return fail(QMM_ERR_INVALID_ARG, "qmm_gemv_batch: null problem list");
    for (int i = 0; i < count; ++i) {
        const qmm_gemv_problem& q = problems[i];
        qmm_status s = check_matrix("qmm_gemv_batch", fmt, q.N, q.K);
        if (s != QMM_OK) return s;
        if (q.K > 32768) return fail(QMM_ERR_UNSUPPORTED, "qmm_gemv_batch: problem %d has K=%lld > 32768", i, (long long)q.K);
        if (!q.packed || !q.x_fp16 || !q.y_fp16) return fail(QMM_ERR_INVALID_ARG, "qmm_gemv_batch: problem %d has a null pointer", i);
        if (!aligned(q.packed, 32) || !aligned(q.x_fp16, 16) || !aligned(q.y_fp16, 16))
            return fail(QMM_ERR_ALIGNMENT, "qmm_gemv_batch: problem %d: packed must be 32-byte, x and y 16-byte aligned", i);
    }
    qmm_status s = check_device("qmm_gemv_batch");
    if (s != QMM_OK) return s;
    return launch_gemv_batch(fmt, problems, count, (cudaStream_t)stream, false);
}

size_t qmm_gemm_workspace_bytes(qmm_format fmt, int64_t M, int64_t N, int64_t K)
{
    if (check_matrix("qmm_gemm_workspace_bytes", fmt, N, K) != QMM_OK || M < 0) return 0;
    return gemm_workspace_bytes(fmt, M, N, K);
}

qmm_status qmm_gemm(qmm_format fmt, const void* packed, int64_t N, int64_t K,
                    const uint16_t* X_fp16, int64_t ldx, uint16_t* Y_fp16, int64_t ldy, int64_t M,
                    void* ws, size_t ws_bytes, void* stream)
{
    qmm_status s = check_matrix("qmm_gemm", fmt, N, K);
    if (s != QMM_OK) return s;
    if (M < 0) return fail(QMM_ERR_INVALID_ARG, "qmm_gemm: M=%lld is negative", (long long)M);
    if (M == 0) return QMM_OK;
    if (M > (1 << 20)) return fail(QMM_ERR_UNSUPPORTED, "qmm_gemm: M=%lld > 2^20", (long long)M);
    if (!packed || !X_fp16 || !Y_fp16) return fail(QMM_ERR_INVALID_ARG, "qmm_gemm: null pointer");
    if (ldx < K || ldy < N) return fail(QMM_ERR_SHAPE, "qmm_gemm: ldx=%lld < K or ldy=%lld < N", (long long)ldx, (long long)ldy);
    if (ldx % 8 || ldy % 8) return fail(QMM_ERR_ALIGNMENT, "qmm_gemm: ldx and ldy must be multiples of 8 elements");
    if (!aligned(packed, 32)) return fail(QMM_ERR_ALIGNMENT, "qmm_gemm: packed must be 32-byte aligned");
    if (!aligned(X_fp16, 16) || !aligned(Y_fp16, 16))
        return fail(QMM_ERR_ALIGNMENT, "qmm_gemm: X and Y must be 16-byte aligned");
    const size_t need = gemm_workspace_bytes(fmt, M, N, K);
    if (!ws || ws_bytes < need)
        return fail(QMM_ERR_WORKSPACE, "qmm_gemm: workspace of %zu bytes needed, %zu given", need, ws ? ws_bytes : (size_t)0);
    if (!aligned(ws, 256)) return fail(QMM_ERR_ALIGNMENT, "qmm_gemm: workspace must be 256-byte aligned");
    if ((s = check_device("qmm_gemm")) != QMM_OK) return s;
    return launch_gemm(fmt, packed, N, K, X_fp16, ldx, Y_fp16, ldy, M, ws, (cudaStream_t)stream);
}

qmm_status qmm_gemm_batch(qmm_format fmt, const qmm_gemm_problem* problems, int count, int64_t M, void* stream)
{
    if (count < 0) return fail(QMM_ERR_INVALID_ARG, "qmm_gemm_batch: count=%d is negative", count);
    if (M < 0 || M > 8) return fail(M < 0 ? QMM_ERR_INVALID_ARG : QMM_ERR_UNSUPPORTED, "qmm_gemm_batch: M=%lld outside [0, 8]", (long long)M);
    if (count == 0 || M == 0) return QMM_OK;
    if (!problems) return fail(QMM_ERR_INVALID_ARG, "qmm_gemm_batch: null problem list");
    for (int i = 0; i < count; ++i) {
        const qmm_gemm_problem& q = problems[i];
        qmm_status s = check_matrix("qmm_gemm_batch", fmt, q.N, q.K);
        if (s != QMM_OK) return s;
        if (!q.packed || !q.X_fp16 || !q.Y_fp16) return fail(QMM_ERR_INVALID_ARG, "qmm_gemm_batch: problem %d has a null pointer", i);
        if (q.ldx < q.K || q.ldy < q.N) return fail(QMM_ERR_SHAPE, "qmm_gemm_batch: problem %d: ldx < K or ldy < N", i);
        if (q.ldx % 8 || q.ldy % 8 || q.ldx >= (1LL << 31) || q.ldy >= (1LL << 31))
            return fail(QMM_ERR_ALIGNMENT, "qmm_gemm_batch: problem %d: ldx and ldy must be multiples of 8 elements below 2^31", i);
        if (!aligned(q.packed, 32) || !aligned(q.X_fp16, 16) || !aligned(q.Y_fp16, 16))
            return fail(QMM_ERR_ALIGNMENT, "qmm_gemm_batch: problem %d: packed must be 32-byte, X and Y 16-byte aligned", i);
    }
    qmm_status s = check_device("qmm_gemm_batch");
    if (s != QMM_OK) return s;
    return launch_gemm_small_batch(fmt, problems, count, M, (cudaStream_t)stream);
}

static qmm_status check_moe(const char* who, const qmm_moe_args* a)
{
    if (!a) return fail(QMM_ERR_INVALID_ARG, "%s: null args", who);
    if (a->T < 0 || a->H <= 0 || a->I <= 0 || a->E <= 0 || a->topk <= 0)
        return fail(QMM_ERR_INVALID_ARG, "%s: T=%d H=%d I=%d E=%d topk=%d out of range", who, a->T, a->H, a->I, a->E, a->topk);
    if (a->topk > a->E) return fail(QMM_ERR_SHAPE, "%s: topk=%d exceeds E=%d", who, a->topk, a->E);
    if (a->E > 1024 || a->topk > 32)
        return fail(QMM_ERR_UNSUPPORTED, "%s: E=%d > 1024 or topk=%d > 32", who, a->E, a->topk);
    if ((int64_t)a->T * a->topk > (1 << 22))
        return fail(QMM_ERR_UNSUPPORTED, "%s: T*topk=%lld > 2^22", who, (long long)a->T * a->topk);
    qmm_status s = check_matrix(who, a->fmt, a->I, a->H);
    if (s != QMM_OK) return s;
    if ((s = check_fmt_everywhere(who, a->fmt)) != QMM_OK) return s;
    return check_matrix(who, a->fmt, a->H, a->I);
}

size_t qmm_moe_workspace_bytes(const qmm_moe_args* args)
{
    if (check_moe("qmm_moe_workspace_bytes", args) != QMM_OK) return 0;
    return moe_workspace_bytes(args);
}

static qmm_status moe_entry(const char* who, const qmm_moe_args* a, void* ws, size_t ws_bytes, void* stream, bool route_only)
{
    qmm_status s = check_moe(who, a);
    if (s != QMM_OK) return s;
    if (a->T == 0) return QMM_OK;                               // nothing to do: no tensor or workspace is touched
    if (!a->logits && !a->w_router) return fail(QMM_ERR_INVALID_ARG, "%s: logits and w_router are both null", who);
    if (a->w_router) {
        if (!a->X) return fail(QMM_ERR_INVALID_ARG, "%s: w_router needs X", who);
        if (!aligned(a->w_router, 32) || !aligned(a->router_logits, 16))
            return fail(QMM_ERR_ALIGNMENT, "%s: w_router must be 32-byte, router_logits 16-byte aligned", who);
        if (a->E % 128) return fail(QMM_ERR_UNSUPPORTED, "%s: w_router needs E %% 128 == 0 (got %d)", who, a->E);
        if ((int64_t)a->T * a->topk > 32 || a->T > 32)
            return fail(QMM_ERR_UNSUPPORTED, "%s: the router product is built for decode-sized layers (T * topk <= 32)", who);
    }
    if (!route_only && (!a->X || !a->w_gate || !a->w_up || !a->w_down || !a->out))
        return fail(QMM_ERR_INVALID_ARG, "%s: null tensor pointer", who);
    if (!aligned(a->logits, 16) || !aligned(a->X, 16) || !aligned(a->out, 16) || !aligned(a->w_gate, 32) ||
        !aligned(a->w_up, 32) || !aligned(a->w_down, 32) || !aligned(a->dbg_H, 16) || !aligned(a->dbg_D, 16))
        return fail(QMM_ERR_ALIGNMENT, "%s: tensors must be 16-byte aligned (packed weights 32-byte)", who);
    const size_t need = moe_workspace_bytes(a);
    if (!ws || ws_bytes < need)
        return fail(QMM_ERR_WORKSPACE, "%s: workspace of %zu bytes needed, %zu given", who, need, ws ? ws_bytes : (size_t)0);
    if (!aligned(ws, 256)) return fail(QMM_ERR_ALIGNMENT, "%s: workspace must be 256-byte aligned", who);
    if ((s = check_device(who)) != QMM_OK) return s;
    return launch_moe(a, ws, route_only, (cudaStream_t)stream);
}

qmm_status qmm_moe(const qmm_moe_args* args, void* ws, size_t ws_bytes, void* stream)
{
    return moe_entry("qmm_moe", args, ws, ws_bytes, stream, false);
}

qmm_status qmm_moe_route(const qmm_moe_args* args, void* ws, size_t ws_bytes, void* stream)
{
    return moe_entry("qmm_moe_route", args, ws, ws_bytes, stream, true);
}

qmm_status qmm_status_check(void* ws, void* stream)
{
    if (!ws) return fail(QMM_ERR_INVALID_ARG, "qmm_status_check: null workspace");
    return status_check(ws, (cudaStream_t)stream);
}

size_t qmm_chain_plan_bytes(qmm_format fmt, const qmm_chain_stage* stages, int count)
{
    return chain_plan_bytes(fmt, stages, count);
}

size_t qmm_chain_workspace_bytes(qmm_format fmt, const qmm_chain_stage* stages, int count)
{
    return chain_workspace_bytes(fmt, stages, count);
}

qmm_status qmm_chain_build(qmm_format fmt, const qmm_chain_stage* stages, int count, void* plan, size_t plan_bytes,
                           void* ws, size_t ws_bytes, qmm_chain_info* info, void* stream)
{
    qmm_status s = check_device("qmm_chain_build");
    if (s != QMM_OK) return s;
    return chain_build(fmt, stages, count, plan, plan_bytes, ws, ws_bytes, info, (cudaStream_t)stream);
}

qmm_status qmm_chain_run(const qmm_chain_info* info, void* stream)
{
    qmm_status s = check_device("qmm_chain_run");
    if (s != QMM_OK) return s;
    return chain_run(info, (cudaStream_t)stream);
}

qmm_status qmm_packed_check(qmm_format fmt, const void* packed, int64_t N, int64_t K, void* ws, void* stream)
{
    qmm_status s = check_matrix("qmm_packed_check", fmt, N, K);
    if (s != QMM_OK) return s;
    if (!packed || !ws) return fail(QMM_ERR_INVALID_ARG, "qmm_packed_check: null pointer");
    if (!aligned(packed, 32)) return fail(QMM_ERR_ALIGNMENT, "qmm_packed_check: packed must be 32-byte aligned");
    if (!aligned(ws, 16)) return fail(QMM_ERR_ALIGNMENT, "qmm_packed_check: workspace must be 16-byte aligned");
    if ((s = check_device("qmm_packed_check")) != QMM_OK) return s;
    return launch_packed_check(fmt, packed, N, K, (int*)ws, (cudaStream_t)stream);
}

qmm_status qmm_debug_config(const char* name, const char* value)
{
    if (!name) {                                                // reset every knob
        g_knobs = DebugKnobs{};
        return QMM_OK;
    }
    const bool off = value == nullptr || value[0] == 0 || strcmp(value, "0") == 0;
    if (strcmp(name, "gemv_force") == 0) {
        int w = 0, sp = 0;
        if (off) {
            g_knobs.gemv_warps = g_knobs.gemv_splits = 0;
            return QMM_OK;
        }
        if (sscanf(value, "%d,%d", &w, &sp) != 2 || (w != 8 && w != 16) || sp < 1 || sp > 64)
            return fail(QMM_ERR_INVALID_ARG, "qmm_debug_config: gemv_force wants \"warps,splits\" with warps 8 or 16, 1 <= splits <= 64");
        g_knobs.gemv_warps = w;
        g_knobs.gemv_splits = sp;
        return QMM_OK;
    }
    if (strcmp(name, "gemm_force") == 0) {
        int b = 0, u = 0;
        if (off) {
            g_knobs.gemm_bn = g_knobs.gemm_units = 0;
            return QMM_OK;
        }
        const int got = sscanf(value, "%d,%d", &b, &u);
        if (got < 1 || !(b == 32 || b == 64 || b == 128 || b == 160 || b == 192 || b == 256) || (got == 2 && u < 1))
            return fail(QMM_ERR_INVALID_ARG, "qmm_debug_config: gemm_force wants \"bn[,units]\" with bn in {32,64,128,160,192,256}");
        g_knobs.gemm_bn = b;
        g_knobs.gemm_units = got == 2 ? u : 0;
        return QMM_OK;
    }
    int* flag = strcmp(name, "gemv_no_cluster") == 0    ? &g_knobs.gemv_no_cluster
                : strcmp(name, "gemm_no_tail_cut") == 0 ? &g_knobs.gemm_no_tail_cut
                : strcmp(name, "gemm_no_small") == 0    ? &g_knobs.gemm_no_small
                : strcmp(name, "moe_no_fuse") == 0      ? &g_knobs.moe_no_fuse
                                                        : nullptr;
    if (!flag) return fail(QMM_ERR_INVALID_ARG, "qmm_debug_config: unknown knob \"%s\"", name);
    *flag = off ? 0 : 1;
    return QMM_OK;
}

qmm_status qmm_debug_wait_give_up(void* ws, int64_t limit_cycles, void* stream)
{
    if (!ws) return fail(QMM_ERR_INVALID_ARG, "qmm_debug_wait_give_up: null workspace");
    if (limit_cycles < 1 || limit_cycles > (1LL << 24))
        return fail(QMM_ERR_INVALID_ARG, "qmm_debug_wait_give_up: limit of %lld cycles outside [1, 2^24]", (long long)limit_cycles);
    qmm_status s = check_device("qmm_debug_wait_give_up");
    if (s != QMM_OK) return s;
    return launch_wait_give_up((int*)ws, (long long)limit_cycles, (cudaStream_t)stream);
}

}  // extern "C"
