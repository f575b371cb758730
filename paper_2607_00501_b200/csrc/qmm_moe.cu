// qmm_moe.cu -- top-k mixture-of-experts feed-forward layer on packed weights.
//
// The paper reports its largest prefill gains on mixture-of-experts models
// (Sec. 4.3) and lists "mixture-of-experts specifics" among the things its
// architecture descriptor carries (Sec. 3.1), but gives no algorithm; the
// steps below are this library's definition (see include/qmm.h):
//   route  -> expert offsets + stable permutation by (expert, token) -> gather rows ->
//   grouped gate/up GEMM with SiLU*mul epilogue -> grouped down GEMM ->
//   weighted combine in slot order.
// Nothing synchronises with the host: the token-tile work list of the grouped
// GEMMs is built on the device from the expert offsets.
#include "qmm_gemm_kernel.cuh"
#include "qmm_route.cuh"

namespace qmm {

qmm_status make_x_map(CUtensorMap* map, const uint16_t* X, int64_t rows, int64_t K, int64_t ld, int box_rows);
qmm_status launch_tc_gemm(int fmt, int bn, int na, int epi, bool dense, const CUtensorMap& map, const GemmParams& p,
                          dim3 grid, cudaStream_t st);
int pick_expert_tile(int64_t total_rows, int experts);
qmm_status launch_moe_gemv(int fmt, bool gate_up, const void* w0, const void* w1, int64_t expert_stride,
                           const uint16_t* x, uint16_t* out, const int* perm, const int* topk_idx,
                           int rows, int topk, int N, int K, cudaStream_t st);

bool moe_small_supported(int T, int topk, int H, int I);
qmm_status launch_moe_small(int fmt, const MoeSmallHost& h, bool route_only, cudaStream_t st);
qmm_status launch_gemv_batch(int fmt, const qmm_gemv_problem* probs, int count, cudaStream_t st, bool out_f32);

// Up to this many (token, expert) rows the expert products run as GEMVs (each row streams its expert's
// matrices once); above it, as grouped tensor-core GEMMs (each expert's matrices are read once per layer).
constexpr int kMoeGemvMaxRows = 32;
dim3 persistent_grid(int bn, int na, int64_t tiles);

// ------------------------------------------------------------ workspace

struct MoeWorkspace {
    size_t status, counts, offsets, num_tiles, tile_expert, tile_row0, tile_rows;
    size_t topk_idx, topk_w, perm, inv_perm, xp, hbuf, dbuf, trace, logits, sync, total;
    int bn, max_tiles;
};

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

static MoeWorkspace moe_layout(const qmm_moe_args* a)
{
    MoeWorkspace w;
    const size_t rows = (size_t)a->T * a->topk;
    w.bn = pick_expert_tile((int64_t)rows, a->E);
    w.max_tiles = (int)((rows + w.bn - 1) / w.bn) + a->E;
    size_t o = 0;
    auto take = [&](size_t bytes) { const size_t at = o; o = align_up(o + bytes, 256); return at; };
    w.status = take(256);
    w.counts = take((size_t)a->E * 4);
    w.sync = take((size_t)(w.max_tiles + 3) * 4);          // hand-over of token tiles between the two grouped products (directly after counts: one memset clears both)
    w.num_tiles = take(4);                                 // (counts, hand-over words and this are cleared by one memset per call)
    w.offsets = take((size_t)(a->E + 1) * 4);
    w.tile_expert = take((size_t)w.max_tiles * 4);
    w.tile_row0 = take((size_t)w.max_tiles * 4);
    w.tile_rows = take((size_t)w.max_tiles * 4);
    w.topk_idx = take(rows * 4);
    w.topk_w = take(rows * 4);
    w.perm = take(rows * 4);
    w.inv_perm = take(rows * 4);
    w.xp = take(rows * (size_t)a->H * 2);
    w.hbuf = take(rows * (size_t)a->I * 2);
    w.dbuf = take(rows * (size_t)a->H * 2);
    w.logits = take(a->w_router ? (size_t)a->T * a->E * 4 : 0);   // router logits when the library computes them
    w.trace = take(4096);                                  // pipeline trace of the gate/up GEMM (tuning aid, QMM_GEMM_TRACE)
    w.total = o;
    return w;
}

size_t moe_workspace_bytes(const qmm_moe_args* a) { return moe_layout(a).total; }

// ---------------------------------------------------------------- route

// One warp per token; also counts rows per expert.
template <int MAX_PER_LANE>
__global__ void route_kernel(const float* __restrict__ logits, int T, int E, int topk,
                             int* __restrict__ idx_out, float* __restrict__ w_out,
                             int* __restrict__ idx_user, float* __restrict__ w_user, int* __restrict__ counts)
{
    pdl_launch_dependents();
    pdl_wait();
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= T) return;
    int sel_idx;
    float w;
    route_token<MAX_PER_LANE>(logits + (size_t)warp * E, E, topk, lane, sel_idx, w);
    if (lane < topk) {
        const size_t o = (size_t)warp * topk + lane;
        idx_out[o] = sel_idx;
        w_out[o] = w;
        if (idx_user) idx_user[o] = sel_idx;
        if (w_user) w_user[o] = w;
        atomicAdd(&counts[sel_idx], 1);                   // a count: the order of the adds does not matter
    }
}

// Decode-sized layers (T * topk <= 32): routing, expert offsets and the stable
// permutation in ONE block, so that the layer is four dependent launches.
// Warp t routes token t; then one warp ranks the <= 32 (token, slot) pairs by
// (expert, flat index) and every thread e derives expert_offsets[e].
template <int MAX_PER_LANE>
__global__ void __launch_bounds__(1024)
route_small_kernel(const float* __restrict__ logits, int T, int E, int topk,
                   int* __restrict__ idx_out, float* __restrict__ w_out, int* __restrict__ idx_user, float* __restrict__ w_user,
                   int* __restrict__ offsets, int* __restrict__ offsets_user,
                   int* __restrict__ perm, int* __restrict__ perm_user, int* __restrict__ inv_perm)
{
    pdl_launch_dependents();
    pdl_wait();
    __shared__ int s_e[32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total = T * topk;
    if (warp < T) {
        int sel_idx;
        float w;
        route_token<MAX_PER_LANE>(logits + (size_t)warp * E, E, topk, lane, sel_idx, w);
        if (lane < topk) {
            const int o = warp * topk + lane;
            idx_out[o] = sel_idx;
            w_out[o] = w;
            if (idx_user) idx_user[o] = sel_idx;
            if (w_user) w_user[o] = w;
            s_e[o] = sel_idx;
        }
    }
    __syncthreads();
    if (warp == 0 && lane < total) {                       // rank of pair `lane` in the (expert, flat index) order
        const int mine = s_e[lane];
        int r = 0;
        for (int j = 0; j < total; ++j) {
            const int other = s_e[j];
            r += (other < mine || (other == mine && j < lane)) ? 1 : 0;
        }
        perm[r] = lane;
        if (perm_user) perm_user[r] = lane;
        inv_perm[lane] = r;
    }
    for (int e = threadIdx.x; e <= E; e += blockDim.x) {   // rows of the experts before e
        int c = 0;
        for (int j = 0; j < total; ++j) c += s_e[j] < e ? 1 : 0;
        offsets[e] = c;
        if (offsets_user) offsets_user[e] = c;
    }
}

// One block per expert e (1024 threads).  First the block derives what the
// exclusive scan over the per-expert counts gives expert e -- its first row
// (expert_offsets[e]) and its first token tile -- by summing the counts of the
// experts before it, and writes its entries of the token-tile list of the
// grouped GEMMs.  Then it walks the T*topk (token, slot) pairs in flat order
// (a contiguous run per thread) and appends those routed to e, which yields the
// stable order by (expert, token).  perm[r] = flat index, inv_perm[flat] = r.
constexpr int kPermuteThreads = 1024;
constexpr int kPermutePer = 16;       // (token, slot) pairs per thread and pass

__global__ void __launch_bounds__(kPermuteThreads)
permute_kernel(const int* __restrict__ topk_idx, int total, const int* __restrict__ counts, int E, int bn,
               int* __restrict__ offsets, int* __restrict__ offsets_user, int* __restrict__ num_tiles,
               int* __restrict__ tile_expert, int* __restrict__ tile_row0, int* __restrict__ tile_rows,
               int* __restrict__ perm, int* __restrict__ perm_user, int* __restrict__ inv_perm)
{
    pdl_launch_dependents();
    pdl_wait();
    __shared__ int s_warp[kPermuteThreads / 32];
    __shared__ int s_rows[kPermuteThreads / 32], s_tiles[kPermuteThreads / 32];
    __shared__ int s_base;
    const int e = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // rows and token tiles of the experts before e (E <= 1024: one count per thread)
    // (rows stay in expert order; the token tiles are listed busiest expert first, equal counts by
    // expert index, so that the grouped products start their longest tiles first and end on short ones)
    int rows_before = 0, tiles_before = 0;
    const int mine_c = counts[e];
    if ((int)threadIdx.x < E) {
        const int c = counts[threadIdx.x];
        if ((int)threadIdx.x < e) rows_before = c;
        if (c > mine_c || (c == mine_c && (int)threadIdx.x < e)) tiles_before = (c + bn - 1) / bn;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        rows_before += __shfl_xor_sync(0xFFFFFFFFu, rows_before, off);
        tiles_before += __shfl_xor_sync(0xFFFFFFFFu, tiles_before, off);
    }
    if (lane == 0) {
        s_rows[warp] = rows_before;
        s_tiles[warp] = tiles_before;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int r0 = 0, t0 = 0;
        for (int w = 0; w < kPermuteThreads / 32; ++w) {
            r0 += s_rows[w];
            t0 += s_tiles[w];
        }
        const int mine = counts[e];
        const int nt = (mine + bn - 1) / bn;
        s_base = r0;
        offsets[e] = r0;
        if (offsets_user) offsets_user[e] = r0;
        for (int i = 0; i < nt; ++i) {
            tile_expert[t0 + i] = e;
            tile_row0[t0 + i] = r0 + i * bn;
            tile_rows[t0 + i] = min(bn, mine - i * bn);
        }
        if (e == E - 1) {
            offsets[E] = r0 + mine;
            if (offsets_user) offsets_user[E] = r0 + mine;
        }
        if (t0 + nt > 0) atomicMax(num_tiles, t0 + nt);                   // the expert listed last closes the list (num_tiles is zeroed with the counts)
    }
    __syncthreads();

    // A thread takes kPermutePer consecutive pairs (all loads in flight at once), counts those routed
    // to e, and a block-wide exclusive scan of the counts gives where its matches go.
    for (int pass0 = 0; pass0 < total; pass0 += kPermuteThreads * kPermutePer) {
        const int i0 = pass0 + (int)threadIdx.x * kPermutePer;
        unsigned mask = 0;
        if (i0 + kPermutePer <= total) {
            int4 v[kPermutePer / 4];
#pragma unroll
            for (int q = 0; q < kPermutePer / 4; ++q) v[q] = reinterpret_cast<const int4*>(topk_idx + i0)[q];
#pragma unroll
            for (int q = 0; q < kPermutePer / 4; ++q)
                mask |= (unsigned)(v[q].x == e) << (4 * q) | (unsigned)(v[q].y == e) << (4 * q + 1) |
                        (unsigned)(v[q].z == e) << (4 * q + 2) | (unsigned)(v[q].w == e) << (4 * q + 3);
        } else {
            for (int j = 0; j < kPermutePer; ++j)
                if (i0 + j < total && topk_idx[i0 + j] == e) mask |= 1u << j;
        }
        const int cnt = __popc(mask);
        int incl = cnt;                                                   // inclusive scan inside the warp
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int up = __shfl_up_sync(0xFFFFFFFFu, incl, off);
            if (lane >= off) incl += up;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        int before = 0, all = 0;
#pragma unroll
        for (int w = 0; w < kPermuteThreads / 32; ++w) {
            const int c = s_warp[w];
            if (w < warp) before += c;
            all += c;
        }
        int r = s_base + before + incl - cnt;
        while (mask) {
            const int j = __ffs(mask) - 1;
            mask &= mask - 1;
            perm[r] = i0 + j;
            if (perm_user) perm_user[r] = i0 + j;
            inv_perm[i0 + j] = r;
            ++r;
        }
        __syncthreads();
        if (threadIdx.x == 0) s_base += all;
        __syncthreads();
    }
}

// One warp per permuted row: copy the token's activations into expert order.
__global__ void gather_rows_kernel(const uint16_t* __restrict__ X, const int* __restrict__ perm, int total, int topk,
                                   int H, uint16_t* __restrict__ Xp)
{
    pdl_wait();                                       // first: once the dependents may start, the permutation kernel is
    pdl_launch_dependents();                          // complete, so the grouped product reads the tile list without waiting
    const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (r >= total) return;
    const int t = perm[r] / topk;
    const uint4* src = reinterpret_cast<const uint4*>(X + (size_t)t * H);
    uint4* dst = reinterpret_cast<uint4*>(Xp + (size_t)r * H);
    for (int i = lane; i < H / 8; i += 32) dst[i] = src[i];
}

// out[t, :] = fp16( sum_j p[t, j] * D[inv_perm[t*topk + j], :] ), fp32, j ascending.
// One block per token; each thread owns 8 consecutive columns.
// The layer's last kernel also re-zeroes the words the next call counts in (rows per expert, tile
// counters, hand-over words): every kernel that used them has finished once this one may run, and a
// per-call memset node would sit in front of the routing kernel and keep it from overlapping its predecessor.
__global__ void combine_kernel(const uint16_t* __restrict__ D, const int* __restrict__ inv_perm,
                               const float* __restrict__ topk_w, int topk, int H, uint16_t* __restrict__ out,
                               int* __restrict__ clear_ptr, int clear_n)
{
    pdl_launch_dependents();
    pdl_wait();
    if (blockIdx.x == 0)
        for (int i = threadIdx.x; i < clear_n; i += blockDim.x) clear_ptr[i] = 0;
    const int t = blockIdx.x;
    for (int c = threadIdx.x * 8; c < H; c += blockDim.x * 8) {
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int j = 0; j < topk; ++j) {
            const int r = inv_perm[t * topk + j];
            const float p = topk_w[t * topk + j];
            const uint4 d = *reinterpret_cast<const uint4*>(D + (size_t)r * H + c);
            const __half2* h = reinterpret_cast<const __half2*>(&d);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(h[i]);
                acc[2 * i] = fmaf(p, f.x, acc[2 * i]);
                acc[2 * i + 1] = fmaf(p, f.y, acc[2 * i + 1]);
            }
        }
        uint4 o;
        __half2* oh = reinterpret_cast<__half2*>(&o);
#pragma unroll
        for (int i = 0; i < 4; ++i) oh[i] = __floats2half2_rn(acc[2 * i], acc[2 * i + 1]);
        *reinterpret_cast<uint4*>(out + (size_t)t * H + c) = o;
    }
}

// ------------------------------------------------------------------ host

template <typename... Args>
static cudaError_t launch_pdl(void (*kernel)(Args...), dim3 grid, dim3 block, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

qmm_status launch_moe(const qmm_moe_args* a, void* ws, bool route_only, cudaStream_t st)
{
    const MoeWorkspace w = moe_layout(a);
    uint8_t* base = (uint8_t*)ws;
    int* status = (int*)(base + w.status);
    int* counts = (int*)(base + w.counts);
    int* tile_sync = (int*)(base + w.sync);
    int* offsets = (int*)(base + w.offsets);
    int* num_tiles = (int*)(base + w.num_tiles);
    int* tile_expert = (int*)(base + w.tile_expert);
    int* tile_row0 = (int*)(base + w.tile_row0);
    int* tile_rows = (int*)(base + w.tile_rows);
    int* topk_idx = (int*)(base + w.topk_idx);
    float* topk_w = (float*)(base + w.topk_w);
    int* perm = (int*)(base + w.perm);
    int* inv_perm = (int*)(base + w.inv_perm);
    uint16_t* xp = (uint16_t*)(base + w.xp);
    uint16_t* hbuf = a->dbg_H ? a->dbg_H : (uint16_t*)(base + w.hbuf);
    uint16_t* dbuf = a->dbg_D ? a->dbg_D : (uint16_t*)(base + w.dbuf);
    const int total = a->T * a->topk;

    cudaError_t e;
    const float* logits = a->logits;
    if (a->w_router) {
        // router product: T independent GEMVs of the [E, H] router matrix, fp32 outputs, one launch
        float* lg = a->router_logits ? a->router_logits : (float*)(base + w.logits);
        qmm_gemv_problem probs[32];
        for (int t = 0; t < a->T; ++t) {
            probs[t].packed = a->w_router;
            probs[t].x_fp16 = a->X + (size_t)t * a->H;
            probs[t].y_fp16 = (uint16_t*)(lg + (size_t)t * a->E);
            probs[t].N = a->E;
            probs[t].K = a->H;
        }
        qmm_status s = launch_gemv_batch(a->fmt, probs, a->T, st, true);
        if (s != QMM_OK) return s;
        logits = lg;
    }
    const int per_lane = (a->E + 31) / 32;
    // decode-sized: one block does steps 1-2 and the expert products run as GEMVs
    const bool small = total <= kMoeGemvMaxRows && a->T <= 32 && a->H <= 32768 && a->I <= 32768;
    const size_t gu_stride = (size_t)(a->I / kRowsPerGroup) * (size_t)(a->H / tile_k_of(a->fmt)) * tile_bytes_of(a->fmt);
    const size_t dn_stride = (size_t)(a->H / kRowsPerGroup) * (size_t)(a->I / tile_k_of(a->fmt)) * tile_bytes_of(a->fmt);
    if (small && !g_knobs.moe_no_fuse && moe_small_supported(a->T, a->topk, a->H, a->I)) {
        // decode: the whole layer in two launches (routing inside the gate/up launch, combine inside the down launch)
        MoeSmallHost h;
        h.logits = logits; h.X = a->X; h.w_gate = a->w_gate; h.w_up = a->w_up; h.w_down = a->w_down;
        h.gu_stride = (int64_t)gu_stride; h.dn_stride = (int64_t)dn_stride;
        h.hbuf = hbuf; h.dbg_D = a->dbg_D; h.out = a->out;
        h.T = a->T; h.E = a->E; h.topk = a->topk; h.H = a->H; h.I = a->I;
        h.idx_ws = topk_idx; h.w_ws = topk_w; h.perm_ws = perm; h.inv_ws = inv_perm; h.offsets_ws = offsets;
        h.idx_user = a->topk_idx; h.w_user = a->topk_w; h.perm_user = a->perm; h.offsets_user = a->expert_offsets;
        h.trace = nullptr;
#if defined(QMM_MOE_TRACE) && QMM_MOE_TRACE
        h.trace = (long long*)(base + w.trace);
#endif
        return launch_moe_small(a->fmt, h, route_only, st);
    }
    if (small) {
        if (per_lane <= 4)
            e = launch_pdl(route_small_kernel<4>, dim3(1), dim3(1024), st, logits, (int)a->T, (int)a->E, (int)a->topk, topk_idx,
                           topk_w, a->topk_idx, a->topk_w, offsets, a->expert_offsets, perm, a->perm, inv_perm);
        else
            e = launch_pdl(route_small_kernel<32>, dim3(1), dim3(1024), st, logits, (int)a->T, (int)a->E, (int)a->topk, topk_idx,
                           topk_w, a->topk_idx, a->topk_w, offsets, a->expert_offsets, perm, a->perm, inv_perm);
        if (e != cudaSuccess) return check_cuda(e, "qmm_moe route launch");
    } else {
        // counts, tile counters, hand-over words and the tile count start at zero: the workspace was zero-filled
        // once by the caller and every complete call leaves them zero again (combine_kernel); a routing-only
        // call has no last kernel of that kind and clears them itself, before and after
        if (route_only) {
            e = cudaMemsetAsync(counts, 0, (w.num_tiles - w.counts) + 4, st);
            if (e != cudaSuccess) return check_cuda(e, "qmm_moe clear counts");
        }
        // 1. routing
        const int warps_per_block = 8;
        const dim3 grid((a->T + warps_per_block - 1) / warps_per_block), block(warps_per_block * 32);
        if (per_lane <= 4)
            e = launch_pdl(route_kernel<4>, grid, block, st, a->logits, (int)a->T, (int)a->E, (int)a->topk, topk_idx, topk_w,
                           a->topk_idx, a->topk_w, counts);
        else
            e = launch_pdl(route_kernel<32>, grid, block, st, a->logits, (int)a->T, (int)a->E, (int)a->topk, topk_idx, topk_w,
                           a->topk_idx, a->topk_w, counts);
        if (e != cudaSuccess) return check_cuda(e, "qmm_moe route launch");
        // 2. expert offsets, token-tile list and stable permutation (one block per expert)
        e = launch_pdl(permute_kernel, dim3(a->E), dim3(kPermuteThreads), st, (const int*)topk_idx, total, (const int*)counts,
                       (int)a->E, w.bn, offsets, a->expert_offsets, num_tiles, tile_expert, tile_row0, tile_rows, perm, a->perm,
                       inv_perm);
        if (e != cudaSuccess) return check_cuda(e, "qmm_moe permute launch");
    }
    if (route_only) {
        if (!small) {
            e = cudaMemsetAsync(counts, 0, (w.num_tiles - w.counts) + 4, st);
            if (e != cudaSuccess) return check_cuda(e, "qmm_moe clear counts");
        }
        return QMM_OK;
    }

    if (small) {
        // decode: a few rows -> GEMV path (gate/up with SiLU*mul, down), then the combine
        qmm_status s = launch_moe_gemv(a->fmt, true, a->w_gate, a->w_up, (int64_t)gu_stride, a->X, hbuf, perm, topk_idx, total,
                                       (int)a->topk, (int)a->I, (int)a->H, st);
        if (s != QMM_OK) return s;
        s = launch_moe_gemv(a->fmt, false, a->w_down, nullptr, (int64_t)dn_stride, hbuf, dbuf, perm, topk_idx, total,
                            (int)a->topk, (int)a->H, (int)a->I, st);
        if (s != QMM_OK) return s;
        e = launch_pdl(combine_kernel, dim3(a->T), dim3(256), st, (const uint16_t*)dbuf, (const int*)inv_perm,
                       (const float*)topk_w, (int)a->topk, (int)a->H, a->out, (int*)nullptr, 0);
        if (e != cudaSuccess) return check_cuda(e, "qmm_moe combine launch");
        return QMM_OK;
    }

    // 3. gather rows into expert order
    e = launch_pdl(gather_rows_kernel, dim3((total + 7) / 8), dim3(256), st, a->X, (const int*)perm, total, (int)a->topk,
                   (int)a->H, xp);
    if (e != cudaSuccess) return check_cuda(e, "qmm_moe gather launch");

    // 4. grouped gate/up GEMM with SiLU*mul epilogue -> Hm [total, I]
    {
        CUtensorMap map;
        qmm_status s = make_x_map(&map, xp, total, a->H, a->H, w.bn);
        if (s != QMM_OK) return s;
        GemmParams p = {};
        p.w[0] = (const uint8_t*)a->w_gate;
        p.w[1] = (const uint8_t*)a->w_up;
        p.w_expert_stride = (int64_t)gu_stride;
        p.N = a->I;
        p.K = a->H;
        p.out = hbuf;
        p.ldo = a->I;
        p.a_col_offset = 0;
        p.M = total;
        p.tile_expert = tile_expert;
        p.tile_row0 = tile_row0;
        p.tile_rows = tile_rows;
        p.num_tiles = num_tiles;
        p.status = status;
        p.sync = tile_sync + 2;
        p.sync_signal = 1;
        p.list_ready = 1;
        if (!g_knobs.moe_no_fuse) p.tile_counter = tile_sync;
#if QMM_GEMM_TRACE
        p.trace = (long long*)(base + w.trace);                            // tuning builds only
#endif
        s = launch_tc_gemm(a->fmt, w.bn, 2, kEpiSiluMul, false, map, p, persistent_grid(w.bn, 2, 0), st);
        if (s != QMM_OK) return s;
    }
    // 5. grouped down GEMM -> D [total, H]
    {
        CUtensorMap map;
        qmm_status s = make_x_map(&map, hbuf, total, a->I, a->I, w.bn);
        if (s != QMM_OK) return s;
        const int na = (a->H % 256 == 0) ? 2 : 1;
        GemmParams p = {};
        p.w[0] = (const uint8_t*)a->w_down;
        p.w[1] = na == 2 ? (const uint8_t*)a->w_down + dn_stride / 2 : nullptr;
        p.w_expert_stride = (int64_t)dn_stride;
        p.N = a->H;
        p.K = a->I;
        p.out = dbuf;
        p.ldo = a->H;
        p.a_col_offset = a->H / 2;
        p.M = total;
        p.tile_expert = tile_expert;
        p.tile_row0 = tile_row0;
        p.tile_rows = tile_rows;
        p.num_tiles = num_tiles;
        p.status = status;
        if (!g_knobs.moe_no_fuse) {
            p.sync = tile_sync + 2;
            p.sync_need = (a->I / 128) * GemmGeom<128, 2, kEpiSiluMul, QMM_Q4>::kEpiWarps;   // weight tiles x epilogue warps of the gate/up product
            p.tile_counter = tile_sync + 1;
        }
        s = launch_tc_gemm(a->fmt, w.bn, na, kEpiStore, false, map, p, persistent_grid(w.bn, na, 0), st);
        if (s != QMM_OK) return s;
    }
    // 6. weighted combine
    e = launch_pdl(combine_kernel, dim3(a->T), dim3(256), st, (const uint16_t*)dbuf, (const int*)inv_perm, (const float*)topk_w,
                   (int)a->topk, (int)a->H, a->out, counts, (int)((w.num_tiles - w.counts) / 4 + 1));
    if (e != cudaSuccess) return check_cuda(e, "qmm_moe combine launch");
    return QMM_OK;
}

}  // namespace qmm
