/*
 * qmm.h -- C ABI of libqmm: fused dequantise-and-multiply of block-quantised
 * weights (Q4 / Q8, 32-element blocks along K, one fp16 scale per block) by
 * fp16 activations, for NVIDIA B200 (sm_100a) only.
 *
 * The operations follow the paper's statement of the problem: weights stay in
 * their quantised storage format and are dequantised inside the inner loop of
 * the product instead of being materialised (Sec. 3.3); decode is the M = 1
 * matrix-vector product, prefill the same product on [seq_len x dim]
 * activations (Sec. 3.3, Sec. 3.4); the runtime is reached through a C API,
 * allocates nothing on the hot path and reports errors through a static
 * thread-local buffer (Sec. 3, Sec. 3.2).  The paper gives no block layout, no
 * quantisation formula and no mixture-of-experts algorithm; those conventions
 * are stated here.
 *
 * Conventions for every call
 *   - W is [N, K]: N output features, K input features.  y = W x, Y = X W^T.
 *   - "device" pointers are CUDA device allocations owned by the caller on the
 *     current device; "host" pointers are ordinary host memory.  The library
 *     never allocates or frees device memory and never keeps a pointer after
 *     the call's work has run.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Calls only enqueue work on it and return; they do not synchronise
 *     (qmm_status_check is the exception).
 *   - Arguments are checked on the host before anything is launched.  On
 *     failure nothing is enqueued, a qmm_status other than QMM_OK is returned
 *     and qmm_last_error() describes the problem.
 *   - Supported shapes: K a multiple of 256, N a multiple of 128, M >= 1
 *     (M = 0 / T = 0 is accepted and does nothing).  Other shapes return
 *     QMM_ERR_UNSUPPORTED.  There is no CPU fallback and no other GPU target.
 *   - Device pointers must be 16-byte aligned; packed weight buffers 32-byte.
 *   - Workspaces of qmm_gemm and qmm_moe start with a status word, and qmm_moe
 *     keeps counters in its workspace that every complete call leaves at zero:
 *     zero-fill a workspace once after allocating it, and again after a call on
 *     it was reported as failed (qmm_status_check) or was abandoned midway.
 *   - Packed weights are read before the product kernels wait for the work
 *     that precedes them in the stream (their loads overlap the tail of the
 *     previous kernel).  A packed buffer must therefore be complete when a
 *     product call that reads it is enqueued: written by qmm_pack, a copy or
 *     any ordinary kernel earlier in the same stream is fine; a kernel that
 *     triggers programmatic dependent launch before it has written the
 *     weights is not.
 *
 * Canonical block format (what qmm_pack reads)
 *   Q4 block, 18 bytes: uint16 d (fp16 bits, little endian), uint8 qs[16];
 *     element i of the block has code q_i in [-8, 7] stored as u_i = q_i + 8,
 *     qs[j] = u_{2j} | (u_{2j+1} << 4).
 *   Q8 block, 34 bytes: uint16 d, int8 qs[32] (two's complement).
 *   Q5 block, 22 bytes: uint16 d, uint8 qh[4], uint8 qs[16]; code q_i in
 *     [-16, 15] stored as u_i = q_i + 16: qs as in Q4 with u_i & 15, bit i of the
 *     little-endian 32-bit word qh = u_i >> 4.
 *   Q6 block, 26 bytes: uint16 d, uint8 qh[8], uint8 ql[16]; code q_i in
 *     [-32, 31] stored as u_i = q_i + 32: ql as in Q4 with u_i & 15, bits
 *     2 (i % 4), 2 (i % 4) + 1 of qh[i / 4] = u_i >> 4.
 *   (The paper's kernel library spans 2-bit to 16-bit formats, Sec. 3.3 and
 *   Sec. 4.1; Q5 and Q6 are built for qmm_pack, qmm_dequant, qmm_packed_check,
 *   qmm_gemv, qmm_gemv_static, qmm_gemv_batch, qmm_gemm and qmm_gemm_batch -- every other call returns
 *   QMM_ERR_UNSUPPORTED for them.)
 *   Row n of W holds K/32 consecutive blocks; rows are consecutive; block b of
 *   row n covers k in [32 b, 32 b + 32).  Weight value: float(d) * q (exact in
 *   fp32).  Scales must be finite.
 *
 * Accuracy.  With y_ref and sum|w x| evaluated exactly, every output of every
 * product satisfies |y - y_ref| <= 2e-3 * sum_k |w_k x_k| + 1e-5 (outputs are
 * fp16: an exact result beyond 65504 in magnitude is stored as infinity).  The GEMVs
 * (qmm_gemv*, decode-sized qmm_moe) multiply integer codes by activations
 * exactly and apply the scale in fp32, so this holds for every finite scale.
 * So does qmm_gemm for M <= 8 (its few-token kernel works the same way).
 * The tensor-core products (qmm_gemm for M > 8, qmm_moe with more than 32
 * token-expert rows) feed each weight to the tensor core as fp16(float(d) * q),
 * which adds two limits:
 *   - |d| * max|q| must stay below 65504 (|d| < 8188 for Q4, < 511.75 for Q8),
 *     else the weight becomes inf; qmm_packed_check reports such scales;
 *   - a weight with |d * q| < 2^-14 is a subnormal fp16 and carries an absolute
 *     error of up to 2^-25 instead of a relative one, so the bound becomes
 *     2e-3 * sum|w x| + 1e-5 + 2^-25 * sum_k |x_k| over such weights (scales of
 *     N(0, 0.02) data are >= 1.8e-4: the extra term never applies to them).
 */
#ifndef QMM_H
#define QMM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    QMM_OK = 0,
    QMM_ERR_INVALID_ARG = 1,   /* null pointer, unknown format, negative size           */
    QMM_ERR_SHAPE = 2,         /* K % 32 != 0, ld < row length, topk > E, ...           */
    QMM_ERR_ALIGNMENT = 3,     /* a device pointer or leading dimension is misaligned   */
    QMM_ERR_WORKSPACE = 4,     /* workspace missing or smaller than *_workspace_bytes   */
    QMM_ERR_UNSUPPORTED = 5,   /* valid problem outside what the kernels cover          */
    QMM_ERR_CUDA = 6,          /* a CUDA runtime/driver call failed (message has it)    */
    QMM_ERR_DEVICE_TIMEOUT = 7,/* a bounded wait inside a kernel gave up                */
    QMM_ERR_BAD_WEIGHTS = 8    /* qmm_packed_check: not a packed buffer of that format  */
} qmm_status;

typedef enum { QMM_Q4 = 4, QMM_Q5 = 5, QMM_Q6 = 6, QMM_Q8 = 8 } qmm_format;

/* Description of the last failure on the calling thread.  Points into a static
 * thread-local buffer (Sec. 3.2: error handling without allocation); never
 * NULL; valid until the next failing call on the same thread.               */
const char* qmm_last_error(void);

/* Library version, major * 10000 + minor * 100 + patch (the paper's runtime is
 * reached through a versioned C API, Sec. 3).                               */
int qmm_version(void);

/* Bytes of the canonical block stream for W[N,K]: N * (K/32) * 18 (Q4), 22
 * (Q5), 26 (Q6) or 34 (Q8).  0 if the arguments are invalid.  (Size queries exist so that the
 * caller can allocate everything up front and the hot path allocates
 * nothing, Sec. 3.2.)                                                       */
size_t qmm_canonical_bytes(qmm_format fmt, int64_t N, int64_t K);

/* Bytes of the device layout produced by qmm_pack (opaque, position
 * independent, copyable with cudaMemcpy; packed buffers of matrices with the
 * same K may be concatenated to form the packed buffer of the row-wise
 * concatenated matrix).  0 if the arguments are invalid or unsupported.     */
size_t qmm_packed_bytes(qmm_format fmt, int64_t N, int64_t K);

/* Repack canonical blocks into the device layout (the analogue of the paper's
 * offline conversion into its native weight format, Sec. 3 / Sec. 4.1).  Off
 * the hot path; integer and bit moves only.
 *   canonical  device, qmm_canonical_bytes(fmt,N,K) bytes, read only
 *   packed     device, qmm_packed_bytes(fmt,N,K) bytes, written            */
qmm_status qmm_pack(qmm_format fmt, const void* canonical, int64_t N, int64_t K,
                    void* packed, void* stream);

/* Validation aid: device layout -> fp32 W[N,K] row-major, w = float(d) * q --
 * the materialised weights that the fused kernels never write (Sec. 3.3
 * describes dequantisation inside the product's inner loop instead).
 *   packed  device, read only;  w_out  device, N*K floats, written.        */
qmm_status qmm_dequant(qmm_format fmt, const void* packed, int64_t N, int64_t K,
                       float* w_out, void* stream);

/* Plausibility check of a packed buffer (off the hot path; the product calls
 * themselves cannot tell a packed buffer from other bytes, because the device
 * layout has no header: packed_bytes == canonical_bytes, and buffers
 * concatenate).  A kernel looks at every scale where the layout of `fmt` and
 * [N, K] puts it; if one is inf / NaN or at least 65504 / max|q| in magnitude
 * (see "Accuracy" above) it writes QMM_ERR_BAD_WEIGHTS to the status word at
 * the start of `ws`, which the next qmm_status_check(ws, stream) returns.
 * Canonical bytes passed as packed, or a buffer of the other format, put code
 * bytes where scales belong and fail within a few hundred values; a buffer
 * that passes has finite, tensor-core-safe scales and nothing more is implied.
 * The paper's loader validates a converted model file once at load time
 * (Sec. 3.1); this is the same step for one matrix.
 *   packed  device, read only;  ws  device, >= 16 bytes, zeroed once (any
 *   qmm_gemm / qmm_moe workspace will do).                                  */
qmm_status qmm_packed_check(qmm_format fmt, const void* packed, int64_t N, int64_t K,
                            void* ws, void* stream);

/* Decode matrix-vector product (Sec. 3.3, "GEMV (decode, M=1)"):
 *   y[n] = fp16( sum_b float(d[n,b]) * sum_{i<32} q[n,b,i] * x[32 b + i] ),
 * accumulated in fp32.  When N is too small to occupy the GPU the K range is
 * split across thread blocks and their sums are added in a fixed order:
 * inside a thread-block cluster through shared memory, or (more than 8
 * splits) through fp32 partial sums in the workspace and a second stage.
 *   packed    device, from qmm_pack, read only
 *   x_fp16    device, K fp16 values (bit patterns), read only
 *   y_fp16    device, N fp16 values, written
 *   ws        device, at least qmm_gemv_workspace_bytes(fmt,N,K) bytes; may be
 *             NULL when that size is 0, which it is whenever the K split (if
 *             any) fits a cluster.  Contents are scratch.  (The size query
 *             follows Sec. 3.2: all memory is obtained before the hot path.) */
size_t qmm_gemv_workspace_bytes(qmm_format fmt, int64_t N, int64_t K);
qmm_status qmm_gemv(qmm_format fmt, const void* packed, int64_t N, int64_t K,
                    const uint16_t* x_fp16, uint16_t* y_fp16,
                    void* ws, size_t ws_bytes, void* stream);

/* Several independent decode products in one launch: y_i = W_i x_i for
 * i < count, all in format fmt (Sec. 3.3: fusing what other runtimes dispatch
 * as separate kernels matters most in decode, where each kernel is short).
 * The products must be independent: every x_i is ready when the call's work
 * starts, no y_i is another problem's input.  Shapes may differ.  Results are
 * those of qmm_gemv up to the order of the fp32 additions.  No workspace.
 *   problems  HOST array of `count` descriptors (read during the call only);
 *             the pointers inside are device pointers with the alignment
 *             rules of qmm_gemv; K <= 32768.                                */
typedef struct {
    const void* packed;        /* device, from qmm_pack                        */
    const uint16_t* x_fp16;    /* device, K fp16 values                        */
    uint16_t* y_fp16;          /* device, N fp16 values, written               */
    int64_t N, K;
} qmm_gemv_problem;
qmm_status qmm_gemv_batch(qmm_format fmt, const qmm_gemv_problem* problems, int count, void* stream);

/* Front half of a gated feed-forward block for one token, in one launch:
 *     h[n] = fp16( silu(g[n]) * u[n] ),  g = W_gate x,  u = W_up x,
 * g and u accumulated in fp32 and never rounded or written (the paper fuses
 * operator sequences within the feed-forward block to save launches and
 * round trips through memory, Sec. 3.3; it does not spell out which).
 * silu(g) = g / (1 + exp(-g)).  W_gate and W_up are [N, K], packed separately.
 *   packed_gate, packed_up  device, 32-byte aligned
 *   x_fp16  device, [K] fp16;  h_fp16  device, [N] fp16, written
 * K <= 32768.  No workspace.                                                 */
qmm_status qmm_gemv_gate_up(qmm_format fmt, const void* packed_gate, const void* packed_up,
                            int64_t N, int64_t K, const uint16_t* x_fp16, uint16_t* h_fp16,
                            void* stream);

/* qmm_gemv for callers that cannot allocate.  The paper has no counterpart to
 * this call; it exists for integrations that are not allowed to obtain device
 * memory at the time they need a product: code that runs after a host
 * application has handed out its whole device-memory budget, code that runs
 * under a lock or inside a latency-critical loop where the device-wide
 * synchronisation of an allocation is not acceptable, and plug-ins whose host
 * forbids any allocator call after start-up.  Such a caller has nowhere to
 * get the split-K workspace of qmm_gemv from, so this variant keeps that
 * scratch inside the library: a fixed array of QMM_GEMV_STATIC_SCRATCH_BYTES
 * that every GPU which loads the library holds until the process exits.
 *   - Same arguments and result as qmm_gemv, minus the workspace.  The caller
 *     still owns packed, x_fp16 and y_fp16 (device pointers).
 *   - Shapes whose split-K partial sums need more than the built-in scratch are
 *     rejected with QMM_ERR_WORKSPACE (nothing is enqueued); use qmm_gemv.
 *   - The call allocates nothing and frees nothing, on the host or the device.
 *   - The first call on each device looks up the device address of the scratch
 *     (one runtime query, no allocation by this library).  If the CUDA runtime
 *     loads modules lazily, that first use is also when it places the
 *     library's image -- this array included -- on the device, which can fail
 *     for lack of memory like any module load.  Make that first call outside
 *     any stream capture, e.g. once at start-up on every device that will be
 *     used.
 *   - All calls on a device share the one scratch array, and it keeps whatever
 *     the last call left in it.  The kernels overwrite every element they later
 *     read, so nothing needs clearing, but two calls whose kernels can overlap
 *     on the GPU (different streams, or graphs replayed concurrently) race on
 *     it: keep calls to this function on one device ordered on one stream.   */
#define QMM_GEMV_STATIC_SCRATCH_BYTES (1 << 20)
qmm_status qmm_gemv_static(qmm_format fmt, const void* packed, int64_t N, int64_t K,
                           const uint16_t* x_fp16, uint16_t* y_fp16, void* stream);

/* A whole list of decode products -- dependent or not -- as ONE launch.
 *
 * The paper's decode loop prepares its dispatches once and replays them with
 * nothing allocated and nothing decided on the hot path (Sec. 3.2), and fuses
 * what other runtimes dispatch separately because a kernel per short product is
 * what bounds decode (Sec. 3.3, Sec. 4.2).  Here a decode step's products are
 * described once as a list of stages; stage i computes
 *     QMM_CHAIN_LINEAR        y_i = fp16( W x )                     W [N, K]
 *     QMM_CHAIN_GATE_UP_SILU  y_i = fp16( silu(W_gate x) * (W_up x) ),
 *                              silu(g) = g / (1 + exp(-g)), W_gate, W_up [N, K]
 * (fp32 accumulation) on x = a caller vector (x_stage < 0) or elements
 * [x_offset, x_offset + K) of the output of an earlier stage -- the value as
 * rounded to fp16, exactly what a separate qmm_gemv would have been given.
 * Stages whose inputs are ready together run side by side; a stage that cannot
 * occupy the GPU by its rows alone is cut along K, its partial sums added in a
 * fixed order (same bits on every call).
 *
 * qmm_chain_build (set-up; synchronises `stream`; allocates host memory only)
 * plans the work of every thread block, writes the plan into the caller's
 * device buffer, clears the workspace and fills `info`.  qmm_chain_run is the
 * hot-path call: one cooperative launch, no allocation, no synchronisation.
 *   - plan: device, >= qmm_chain_plan_bytes; ws: device, >=
 *     qmm_chain_workspace_bytes; both 256-byte aligned.  The plan holds
 *     addresses inside `ws`, of the weights and of the x_fp16 / y_fp16 vectors:
 *     all must stay where they are while the plan is used.  The workspace
 *     starts with a status word (qmm_status_check(ws, stream) reports a
 *     give-up of a bounded wait; after one, clear the workspace and rebuild).
 *   - Launches that use one workspace must not overlap on the GPU.
 *   - K <= 32768, K % 256 == 0, N % 128 == 0, x_offset % 8 == 0, <= 4096 stages.
 *   - The launch needs every SM of the device for itself (one block per SM
 *     must be resident at once); it fails with QMM_ERR_CUDA if that cannot be.
 *   - y_fp16 (optional, device, [N] fp16) receives a plain copy of a stage's
 *     output; outputs of stages without it stay internal.                     */
typedef enum { QMM_CHAIN_LINEAR = 0, QMM_CHAIN_GATE_UP_SILU = 1 } qmm_chain_op;
typedef struct {
    int32_t op;                /* qmm_chain_op                                          */
    int32_t x_stage;           /* < 0: x_fp16 below; else the index of an earlier stage */
    int64_t x_offset;          /* first element of that stage's output used as x[0]     */
    const uint16_t* x_fp16;    /* device, [K] fp16, ready when the launch starts        */
    const void* packed;        /* device, from qmm_pack: W, or W_gate                   */
    const void* packed_up;     /* device: W_up (QMM_CHAIN_GATE_UP_SILU), else NULL      */
    int64_t N, K;
    uint16_t* y_fp16;          /* device, [N] fp16, optional                            */
} qmm_chain_stage;
typedef struct {               /* filled by qmm_chain_build; plain data, may be copied  */
    int32_t magic, fmt, stages, grid, threads, smem_bytes;
    uint64_t plan_bytes, ws_bytes;
    void* plan;
    void* ws;
} qmm_chain_info;
size_t qmm_chain_plan_bytes(qmm_format fmt, const qmm_chain_stage* stages, int count);       /* host array */
size_t qmm_chain_workspace_bytes(qmm_format fmt, const qmm_chain_stage* stages, int count);
qmm_status qmm_chain_build(qmm_format fmt, const qmm_chain_stage* stages, int count,
                           void* plan, size_t plan_bytes, void* ws, size_t ws_bytes,
                           qmm_chain_info* info, void* stream);
qmm_status qmm_chain_run(const qmm_chain_info* info, void* stream);

/* Prefill matrix-matrix product (Sec. 3.3 "GEMM (prefill, M>1)", Sec. 3.4):
 *   Y[m,n] = fp16( sum_k w[n,k] * X[m,k] ), fp32 accumulation on the tensor
 * cores; weights enter the contraction as fp16(float(d) * q).
 * For M <= 8 (a decode step of a small batch, the tail of a prefill chunk) the
 * product is bound by streaming W once, like decode (Sec. 3.3), and runs on a
 * kernel of the decode family instead: integer codes times activations on the
 * warp-level tensor path, scales applied in fp32, no workspace use; row m of Y
 * is then the same bits whatever the other rows hold and whatever M in 3..8 is
 * (M = 1 and M = 2 run on the qmm_gemv kernel -- two tokens cost little more
 * than one there -- and give each row the bits of qmm_gemv).
 *   X_fp16  device, [M, ldx] fp16 row-major, ldx >= K, ldx % 8 == 0
 *   Y_fp16  device, [M, ldy] fp16 row-major, ldy >= N, ldy % 8 == 0, written
 *   ws      device, at least qmm_gemm_workspace_bytes(...) bytes: the status
 *           word and, for shapes whose output tiles (or the tiles of their
 *           last round) do not occupy the SMs, the fp32 partial sums of the
 *           pieces the K range of those tiles is cut into (added in a fixed
 *           order by a second kernel, so results are the same bits on every
 *           call).  8 KB for most shapes, up to two slots of one output tile
 *           per SM (39 MB) where tiles are cut.  (Size query: Sec. 3.2.)     */
size_t qmm_gemm_workspace_bytes(qmm_format fmt, int64_t M, int64_t N, int64_t K);
qmm_status qmm_gemm(qmm_format fmt, const void* packed, int64_t N, int64_t K,
                    const uint16_t* X_fp16, int64_t ldx,
                    uint16_t* Y_fp16, int64_t ldy, int64_t M,
                    void* ws, size_t ws_bytes, void* stream);

/* Many independent few-token products in one launch: problem i computes
 *   Y_i[m,n] = fp16( sum_k w_i[n,k] * X_i[m,k] ),  m < M,  1 <= M <= 8 for all,
 * i.e. every matrix of a decode step for a batch of up to eight sequences (the
 * paper's decode gains come from fewer, fused dispatches, Sec. 3.3; decode is
 * bound by streaming the weights, which this launch does once for all M
 * tokens).  The products must be independent, as for qmm_gemv_batch.  Integer
 * codes times activations, scales applied in fp32 (the accuracy of the GEMVs);
 * row m of Y_i does not depend on the other rows, nor on M within 3..8 (one and
 * two tokens run on the single-token batched kernel: two tokens cost little
 * more than one there).  No workspace.
 *   problems  HOST array of `count` descriptors (read during the call only);
 *             pointers inside are device pointers: packed 32-byte aligned,
 *             X [M, ldx] and Y [M, ldy] fp16 row-major, 16-byte aligned,
 *             ldx >= K, ldy >= N, both multiples of 8 and below 2^31.         */
typedef struct {
    const void* packed;        /* device, from qmm_pack                        */
    const uint16_t* X_fp16;    /* device, [M, ldx] fp16                        */
    uint16_t* Y_fp16;          /* device, [M, ldy] fp16, written               */
    int64_t N, K, ldx, ldy;
} qmm_gemm_problem;
qmm_status qmm_gemm_batch(qmm_format fmt, const qmm_gemm_problem* problems, int count, int64_t M, void* stream);

/* Top-k mixture-of-experts feed-forward layer.  The paper names
 * mixture-of-experts models as the case with its largest prefill gains
 * (Sec. 4.3) but gives no algorithm; this library defines it as
 *   1. routing: per token the topk largest router logits, larger first, equal
 *      logits -> lower expert index first; weights = softmax over the selected
 *      logits (fp32);
 *   2. permutation: the T*topk (token, slot) pairs sorted by (expert, token);
 *      perm[r] = t*topk + j, expert_offsets[e] = first sorted row of expert e;
 *   3. per expert e on its rows: G = X Wgate_e^T, U = X Wup_e^T,
 *      Hm = fp16(silu(G) * U) with silu(g) = g / (1 + exp(-g));
 *   4. D = fp16(Hm Wdown_e^T);
 *   5. out[t,:] = fp16( sum_{j<topk} p[t,j] * D[row(t,j),:] ), fp32, j ascending.
 * All pointers are device pointers.                                          */
typedef struct {
    int32_t T, H, I, E, topk;      /* tokens, hidden, expert intermediate, experts, k   */
    int32_t fmt;                   /* qmm_format of all expert matrices                 */
    const float* logits;           /* [T,E] fp32, finite, read only                     */
    const uint16_t* X;             /* [T,H] fp16, read only                             */
    const void* w_gate;            /* E packed [I,H] matrices, stride packed_bytes(I,H) */
    const void* w_up;              /* same                                              */
    const void* w_down;            /* E packed [H,I] matrices, stride packed_bytes(H,I) */
    uint16_t* out;                 /* [T,H] fp16, written                               */
    int32_t* topk_idx;             /* [T,topk]  optional (NULL = not exported)          */
    float* topk_w;                 /* [T,topk]  optional                                */
    int32_t* perm;                 /* [T*topk]  optional                                */
    int32_t* expert_offsets;       /* [E+1]     optional                                */
    uint16_t* dbg_H;               /* [T*topk, I] fp16 in permuted row order, optional  */
    uint16_t* dbg_D;               /* [T*topk, H] fp16 in permuted row order, optional  */
    /* Optional router product (decode-sized layers, T * topk <= 32, E % 128 == 0): when
     * w_router is non-NULL the logits are computed by the library, logits[t, e] =
     * sum_k W_router[e, k] * X[t, k] accumulated and kept in fp32 (one more fused launch
     * of the decode step, Sec. 3.3), and `logits` above is ignored (may be NULL).     */
    const void* w_router;          /* packed [E, H] matrix in format fmt, or NULL       */
    float* router_logits;          /* [T, E] fp32, optional export of those logits      */
} qmm_moe_args;

/* Workspace size for these arguments (host pointer to args; only the sizes are
 * read).  Obtained once, before the hot path (Sec. 3.2).                     */
size_t qmm_moe_workspace_bytes(const qmm_moe_args* args);
/* Steps 1-5.  ws: device, >= qmm_moe_workspace_bytes(args).                  */
qmm_status qmm_moe(const qmm_moe_args* args, void* ws, size_t ws_bytes, void* stream);
/* Steps 1-2 only; fills the optional routing outputs that are non-NULL.  (The
 * paper lists routing among the mixture-of-experts specifics its architecture
 * descriptor carries, Sec. 3.1, without giving the rule; the rule is above.)  */
qmm_status qmm_moe_route(const qmm_moe_args* args, void* ws, size_t ws_bytes, void* stream);

/* Waits for `stream`, then reports what the kernels that used `ws` recorded in
 * its status word since this call last cleared it: QMM_ERR_DEVICE_TIMEOUT if a
 * bounded wait gave up, QMM_ERR_BAD_WEIGHTS from qmm_packed_check, else QMM_OK.
 * The only call that synchronises; errors otherwise travel through the static
 * thread-local buffer of qmm_last_error (Sec. 3.2).
 *   ws: device workspace of qmm_gemm, qmm_moe or qmm_packed_check.           */
qmm_status qmm_status_check(void* ws, void* stream);

/* ---- debug entry points (tests and tuning; no counterpart in the paper) ----
 *
 * qmm_debug_config sets a process-wide knob that forces a launch geometry;
 * none changes a result beyond the order of fp32 additions.  The library
 * reads no environment variable.  Not synchronised: call it while no other
 * thread is inside the library.  name == NULL resets every knob; value NULL,
 * "" or "0" clears the named one.
 *   "gemv_force"       "warps,splits"  block size (8 | 16 warps) and K split of qmm_gemv
 *   "gemv_no_cluster"  "1"             K split through workspace partial sums + second kernel
 *   "gemm_force"       "bn[,units]"    token tile and (tile, k-block) units per block of qmm_gemm
 *   "gemm_no_tail_cut" "1"             last, partly filled round of tiles left whole
 *   "gemm_no_small"    "1"             M <= 8 through the tensor-core kernel, not the few-token kernel
 *   "moe_no_fuse"      "1"             decode-sized qmm_moe as separate route / product / combine launches
 */
qmm_status qmm_debug_config(const char* name, const char* value);

/* Exercises the give-up path of the kernels' bounded waits without any other
 * work in flight: one warp waits on a barrier that nothing completes for
 * limit_cycles clock cycles (1 .. 2^24, i.e. at most ~10 ms), then records
 * QMM_ERR_DEVICE_TIMEOUT in the status word at the start of ws, as a GEMM
 * kernel whose pipeline stalled would.  The next qmm_status_check(ws, stream)
 * returns it; the context stays usable.  ws: device, >= 16 bytes.           */
qmm_status qmm_debug_wait_give_up(void* ws, int64_t limit_cycles, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* QMM_H */
