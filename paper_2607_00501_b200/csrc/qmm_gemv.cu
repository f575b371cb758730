// qmm_gemv.cu -- decode matrix-vector product y = W x on packed Q4/Q8 weights.
//
// The paper's decode kernels dequantise inside the inner loop so that only the
// quantised bytes cross the memory bus (Sec. 3.3); this is the same idea laid
// out for B200: the kernel is bound by HBM bandwidth on the packed bytes, so
// each lane streams 32-byte code chunks with many loads in flight, expands
// them to exact fp16 integers in registers and accumulates in fp32.
//
// Work decomposition.  A row group is 32 rows, one per lane, so no cross-lane
// reduction is ever needed: every lane owns one output.  A thread block takes
// one (row group, K split) item; its warps share the item's tiles round-robin,
// then add their per-lane partial sums through shared memory in warp order.
// With splits > 1 the block writes fp32 partials [split][N] to the workspace
// and a second kernel adds the splits in ascending order (fixed order, so the
// result does not depend on scheduling).
#include "qmm_common.cuh"
#include "qmm_gemv_core.cuh"
#include "qmm_route.cuh"

#include <stdio.h>

namespace qmm {

#ifndef QMM_GEMV_UNROLL
#define QMM_GEMV_UNROLL 2
#endif
constexpr int kUnroll = QMM_GEMV_UNROLL;   // tile pairs in flight per warp (4 x 1 KiB of codes per warp)

// Thread-block cluster helpers of the split-K form without workspace.
constexpr int kMaxClusterSplits = 8;                            // portable cluster size (room in shared memory)
constexpr int kPlanClusterSplits = 4;                           // what the plan asks for: clusters of 8 measured slower to schedule

// Codes and scales of kUnroll tile pairs held in registers.
template <int FMT>
struct TileRegs {
    u32x8 cp[kUnroll], cq[kUnroll];
    typename HiRegs<FMT>::type hp[kUnroll], hq[kUnroll];          // high bits (Q5 / Q6 only)
    typename ScaleRegs<FMT>::type sp[kUnroll], sq[kUnroll];
};

// grid.x blocks loop over items = (row-group pairs) * splits; block = WARPS warps.
// Dynamic shared memory: K fp16 activations, K fp16 zeros, then WARPS*64 floats.
//
// Weights never depend on the previous kernel in the stream, activations do.
// So each warp issues the loads of its first group *before* waiting for the
// previous kernel (programmatic dependent launch): the HBM latency of one
// product hides behind the tail of the one before it.
//
// K split across blocks (splits > 1), two forms.  With `partial`: fp32 partial sums go to the workspace
// and gemv_reduce_kernel adds them.  Without (partial == nullptr): the `splits` blocks of an item are a
// thread-block cluster; each writes its 64 sums into the shared memory of the cluster's first block
// (distributed shared memory), which adds them in split order after a cluster barrier and writes y --
// no workspace, no second launch, same bits on every call.
//
// GATEUP: the row-group pair of an item is (group j of `packed`, group j of `packed_up`) -- the gate
// rows and the up rows of the same 32 outputs -- and the item writes h = fp16(silu(g) * u) for them
// (no K split across blocks in this form).
//
// TWO: two activation vectors (x and x + ldx2) against the same matrix, outputs to y and y + ldy2.  The
// one-row-per-lane MMA scheme leaves B columns 4..7 zero; the second token rides there (column 4+j = its
// quadruple in slot group j: lanes with g == t + 4 read it), so both products cost the MMAs of one, and
// the lanes with t >= 2, idle otherwise, receive the second token's sums.  Each token's sums are added
// exactly as in the single-token form (cluster form or no K split only).
template <int FMT, int WARPS, bool GATEUP = false, bool TWO = false>
__global__ void __launch_bounds__(WARPS * 32, 768 / (WARPS * 32))
gemv_kernel(const uint8_t* __restrict__ packed, const uint16_t* __restrict__ x,
            uint16_t* __restrict__ y, float* __restrict__ partial,
            int N, int K, int tiles_per_row, int splits, int items, const uint8_t* __restrict__ packed_up,
            int64_t ldx2, int64_t ldy2)
{
    static_assert(!(GATEUP && TWO), "the fused gate/up form takes one token");
    constexpr int NTOK = TWO ? 2 : 1;
    extern __shared__ uint4 smem[];
    uint4* xs = smem;                                           // [NTOK][K / 8]
    uint4* zs = smem + NTOK * (K / 8);
    float* red = reinterpret_cast<float*>(zs + K / 8);          // [WARPS][NTOK][64]
    float* cred = red + WARPS * NTOK * 64;                      // cluster form: [2][kMaxClusterSplits][NTOK * 64] in the first block
    const bool clustered = !GATEUP && splits > 1 && partial == nullptr;
    int cluster_round = 0;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int TB = Fmt<FMT>::tile_bytes;
    constexpr int XV = Fmt<FMT>::tile_k / 8;                    // uint4 of activations per tile
    constexpr int STEP = kUnroll * WARPS;

    const int tps = tiles_per_row / splits;                     // tiles per item
    const size_t group_bytes = (size_t)tiles_per_row * TB;
    const uint8_t* lane_base = packed + 32 * lane;
    // second row group of the pair: the next group of the same matrix, or the same group of the up matrix
    const ptrdiff_t q_delta = GATEUP ? packed_up - packed : (ptrdiff_t)group_bytes;
    constexpr int GROUPS_PER_ITEM = GATEUP ? 1 : 2;

    int item = blockIdx.x;
    int pair = item / splits, s = item - pair * splits;
    int t = s * tps + warp, t_end = (s + 1) * tps;
    const uint8_t* tiles_p = lane_base + (size_t)(GROUPS_PER_ITEM * pair) * group_bytes;

    TileRegs<FMT> r;
    // slot u of the register file holds tile pair t + u * WARPS of the current item
    auto load_slot = [&](int u, int tt) {
        const uint8_t* tp = tiles_p + (size_t)tt * TB;
        const uint8_t* tq = tp + q_delta;
        r.cp[u] = ld_stream_256(tp);
        r.cq[u] = ld_stream_256(tq);
        r.hp[u] = load_hi<FMT>(tp - 32 * lane, lane);
        r.hq[u] = load_hi<FMT>(tq - 32 * lane, lane);
        r.sp[u] = load_scales<FMT>(tp - 32 * lane, lane);
        r.sq[u] = load_scales<FMT>(tq - 32 * lane, lane);
    };
    auto load_group = [&]() {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
            if (t + u * WARPS < t_end) load_slot(u, t + u * WARPS);
    };
    if (item < items) load_group();

    pdl_launch_dependents();
    pdl_wait();                                                 // x may come from the previous kernel
    for (int i = threadIdx.x; i < K / 8; i += WARPS * 32) {
        xs[i] = reinterpret_cast<const uint4*>(x)[i];
        if (TWO) xs[K / 8 + i] = reinterpret_cast<const uint4*>(x + ldx2)[i];
        zs[i] = make_uint4(0u, 0u, 0u, 0u);
    }
    __syncthreads();
    const uint4* xb = ((lane >> 2) == (lane & 3)) ? xs : (TWO && (lane >> 2) == (lane & 3) + 4) ? xs + K / 8 : zs;
    Q4Consts kc;
    kc.init();

    while (item < items) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        while (t < t_end) {
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int tt = t + u * WARPS;
                if (tt < t_end) tile_pair_mma<FMT>(r.cp[u], r.cq[u], r.hp[u], r.hq[u], r.sp[u], r.sq[u], xb + tt * XV, acc, kc);
            }
            t += STEP;
            if (t < t_end) load_group();
        }
        const int done_pair = pair, done_s = s;
        item += gridDim.x;
        if (item < items) {                                     // next item's loads fly during the reduction
            pair = item / splits;
            s = item - pair * splits;
            t = s * tps + warp;
            t_end = (s + 1) * tps;
            tiles_p = lane_base + (size_t)(GROUPS_PER_ITEM * pair) * group_bytes;
            load_group();
        }
        // add the warps' partial sums in warp order
        if (TWO || (lane & 3) < 2) {                            // lanes that received sums (see above)
            const int row = (lane & ~3) + 2 * (lane & 1);
            float* w = red + (warp * NTOK + (TWO ? (lane & 3) >> 1 : 0)) * 64;
            w[row] = acc[0];
            w[row + 1] = acc[1];
            w[32 + row] = acc[2];
            w[32 + row + 1] = acc[3];
        }
        __syncthreads();
        if (GATEUP) {
            if (threadIdx.x < 32) {                             // red[.. 0..31] = gate sums, red[.. 32..63] = up sums
                float g = red[threadIdx.x], up = red[32 + threadIdx.x];
#pragma unroll
                for (int w = 1; w < WARPS; ++w) {
                    g += red[w * 64 + threadIdx.x];
                    up += red[w * 64 + 32 + threadIdx.x];
                }
                y[done_pair * 32 + threadIdx.x] = __half_as_ushort(__float2half_rn((g / (1.0f + expf(-g))) * up));
            }
        } else if (clustered) {
            // every block of the cluster runs the same sequence of items, one split each
            float* slot = cred + (cluster_round & 1) * (kMaxClusterSplits * NTOK * 64);
            if (threadIdx.x < NTOK * 64) {
                float sum = red[threadIdx.x];
#pragma unroll
                for (int w = 1; w < WARPS; ++w) sum += red[w * NTOK * 64 + threadIdx.x];
                st_cluster_rank0(slot + done_s * NTOK * 64 + threadIdx.x, sum);
            }
            cluster_sync();
            if (done_s == 0 && threadIdx.x < NTOK * 64) {
                float total = slot[threadIdx.x];
                for (int sp = 1; sp < splits; ++sp) total += slot[sp * NTOK * 64 + threadIdx.x];
                uint16_t* yt = TWO && threadIdx.x >= 64 ? y + ldy2 : y;
                yt[done_pair * 64 + (threadIdx.x & 63)] = __half_as_ushort(__float2half_rn(total));
            }
            ++cluster_round;                                    // (two slots: the next item's sums do not wait for this read)
        } else if (threadIdx.x < NTOK * 64) {
            float sum = red[threadIdx.x];
#pragma unroll
            for (int w = 1; w < WARPS; ++w) sum += red[w * NTOK * 64 + threadIdx.x];
            const int n = done_pair * 64 + (threadIdx.x & 63);
            if (splits == 1)
                (TWO && threadIdx.x >= 64 ? y + ldy2 : y)[n] = __half_as_ushort(__float2half_rn(sum));
            else
                partial[(size_t)done_s * N + n] = sum;              // (single token only)
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------- batch
//
// Many independent products in ONE launch (fused q/k/v, gate/up, all the
// matrices of a layer whose inputs are ready...).  The paper's decode gains
// come from issuing fewer, fused dispatches (Sec. 3.3); a launch per small
// matrix cannot keep a B200's HBM busy -- a 2 MB matrix is 0.3 us of traffic,
// a launch is several -- so the whole list is streamed by one persistent grid.
//
// Work unit = (problem, pair of row groups): 64 outputs, the block's warps
// split its K range.  The list of units is cut into gridDim.x contiguous
// ranges of equal *cost* (cost of a unit = its number of tiles), so blocks
// finish together although problems differ in K.  No split-K, no workspace.

constexpr int kMaxBatch = 128;

struct BatchProblem {
    const uint8_t* packed;
    const uint16_t* x;
    uint16_t* y;
    const uint16_t* x2;   // TWO form: the second token's activations and outputs
    uint16_t* y2;
    int K;            // input features
    int tpr;          // tiles per row
    int pairs;        // N / 64
    int cost_begin;   // tiles of all earlier problems
};

struct BatchParams {
    int count;
    int total_cost;
    int max_k;
    int out_f32;      // != 0: the y pointers are float*: outputs stay fp32 (router logits)
    BatchProblem p[kMaxBatch];
};

// TWO: every problem has two activation vectors (two decode sequences).  The one-row-per-lane MMA
// scheme leaves B columns 4..7 zero; the second token rides there (column 4+j = its quadruple in slot
// group j: lanes with g == t + 4 read it), so both products cost the MMAs of one, and the lanes with
// t >= 2, idle otherwise, receive the second token's sums (rows 4g+2(t-2), +1 of both row groups).
template <int FMT, int WARPS, bool TWO = false>
#ifndef QMM_BATCH_THREADS_PER_SM
#define QMM_BATCH_THREADS_PER_SM 768
#endif
__global__ void __launch_bounds__(WARPS * 32, QMM_BATCH_THREADS_PER_SM / (WARPS * 32))
gemv_batch_kernel(const __grid_constant__ BatchParams bp)
{
    constexpr int NTOK = TWO ? 2 : 1;
    extern __shared__ uint4 smem[];
    uint4* xs = smem;                                           // [NTOK][max_k / 8]
    uint4* zs = smem + NTOK * (bp.max_k / 8);
    float* red = reinterpret_cast<float*>(zs + bp.max_k / 8);   // [WARPS][NTOK][64]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int TB = Fmt<FMT>::tile_bytes;
    constexpr int XV = Fmt<FMT>::tile_k / 8;
    constexpr int STEP = kUnroll * WARPS;

    // this block's range of the unit list, by cost
    const int c0 = (int)(((long long)bp.total_cost * blockIdx.x) / gridDim.x);
    const int c1 = (int)(((long long)bp.total_cost * (blockIdx.x + 1)) / gridDim.x);
    int pi = 0;
    while (pi < bp.count && bp.p[pi].cost_begin + bp.p[pi].pairs * bp.p[pi].tpr <= c0) ++pi;
    int unit = 0;                                               // pair index within problem pi
    if (pi < bp.count) {
        const int rel = c0 - bp.p[pi].cost_begin;
        unit = rel <= 0 ? 0 : (rel + bp.p[pi].tpr - 1) / bp.p[pi].tpr;
        if (unit >= bp.p[pi].pairs) {
            ++pi;
            unit = 0;
        }
    }
    // a unit belongs to the block whose range holds the unit's first tile
    auto valid = [&](int p, int u) { return p < bp.count && bp.p[p].cost_begin + u * bp.p[p].tpr < c1; };

    TileRegs<FMT> r;
    int t = 0, t_end = 0;
    const uint8_t* tiles_p = nullptr;
    size_t group_bytes = 0;
    auto open_unit = [&](int p, int u) {
        group_bytes = (size_t)bp.p[p].tpr * TB;
        tiles_p = bp.p[p].packed + 32 * lane + (size_t)(2 * u) * group_bytes;
        t = warp;
        t_end = bp.p[p].tpr;
    };
    // slot u of the register file holds tile pair t + u * WARPS of the current item
    auto load_slot = [&](int u, int tt) {
        const uint8_t* tp = tiles_p + (size_t)tt * TB;
        const uint8_t* tq = tp + group_bytes;
        r.cp[u] = ld_stream_256(tp);
        r.cq[u] = ld_stream_256(tq);
        r.hp[u] = load_hi<FMT>(tp - 32 * lane, lane);
        r.hq[u] = load_hi<FMT>(tq - 32 * lane, lane);
        r.sp[u] = load_scales<FMT>(tp - 32 * lane, lane);
        r.sq[u] = load_scales<FMT>(tq - 32 * lane, lane);
    };
    auto load_group = [&]() {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
            if (t + u * WARPS < t_end) load_slot(u, t + u * WARPS);
    };
    bool have = valid(pi, unit);
    if (have) {
        open_unit(pi, unit);
        load_group();
    }

    pdl_launch_dependents();
    pdl_wait();                                                 // activations may come from the previous kernel
    for (int i = threadIdx.x; i < bp.max_k / 8; i += WARPS * 32) zs[i] = make_uint4(0u, 0u, 0u, 0u);
    auto stage_x = [&](int p) {
        for (int i = threadIdx.x; i < bp.p[p].K / 8; i += WARPS * 32) {
            xs[i] = reinterpret_cast<const uint4*>(bp.p[p].x)[i];
            if (TWO) xs[bp.max_k / 8 + i] = reinterpret_cast<const uint4*>(bp.p[p].x2)[i];
        }
    };
    if (have) stage_x(pi);
    __syncthreads();
    const uint4* xb = ((lane >> 2) == (lane & 3)) ? xs : (TWO && (lane >> 2) == (lane & 3) + 4) ? xs + bp.max_k / 8 : zs;
    Q4Consts kc;
    kc.init();

    while (have) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        while (t < t_end) {
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int tt = t + u * WARPS;
                if (tt < t_end) tile_pair_mma<FMT>(r.cp[u], r.cq[u], r.hp[u], r.hq[u], r.sp[u], r.sq[u], xb + tt * XV, acc, kc);
            }
            t += STEP;
            if (t < t_end) load_group();
        }
        const int done_p = pi, done_u = unit;
        if (++unit >= bp.p[pi].pairs) {
            ++pi;
            unit = 0;
        }
        have = valid(pi, unit);
        if (have) {                                             // next unit's loads fly during the reduction
            open_unit(pi, unit);
            load_group();
        }
        if (TWO || (lane & 3) < 2) {
            const int row = (lane & ~3) + 2 * (lane & 1);
            float* w = red + (warp * NTOK + (TWO ? (lane & 3) >> 1 : 0)) * 64;
            w[row] = acc[0];
            w[row + 1] = acc[1];
            w[32 + row] = acc[2];
            w[32 + row + 1] = acc[3];
        }
        __syncthreads();                                        // also: every warp is done with xs
        if (threadIdx.x < 64 * NTOK) {
            float sum = red[threadIdx.x];
#pragma unroll
            for (int w = 1; w < WARPS; ++w) sum += red[w * 64 * NTOK + threadIdx.x];
            uint16_t* yt = TWO && threadIdx.x >= 64 ? bp.p[done_p].y2 : bp.p[done_p].y;
            if (bp.out_f32)
                reinterpret_cast<float*>(yt)[done_u * 64 + (threadIdx.x & 63)] = sum;
            else
                yt[done_u * 64 + (threadIdx.x & 63)] = __half_as_ushort(__float2half_rn(sum));
        }
        if (have && pi != done_p) stage_x(pi);                  // next unit reads other activation vectors
        __syncthreads();
    }
}

// ------------------------------------------------------- MoE decode rows
//
// The expert products of a mixture-of-experts layer when only a few tokens are
// in flight (decode): every permuted row r = (token, expert) is a GEMV against
// its expert's matrices, found on the device from the routing result.
//   GATE_UP: unit = (row r, 32 outputs): the warp's row-group pair is
//            (gate rows, up rows) of the same 32 outputs, so one pass yields
//            G and U; the block writes h = fp16(silu(G) * U).  x = X[token(r)].
//   DOWN:    unit = (row r, 64 outputs) of the down matrix.  x = Hm[r].
struct MoeGemvParams {
    const uint8_t* w0;          // GATE_UP: gate matrices; DOWN: down matrices (expert-major, packed)
    const uint8_t* w1;          // GATE_UP: up matrices
    int64_t expert_stride;      // bytes between experts
    const uint16_t* x;          // GATE_UP: X [T, K]; DOWN: Hm [rows, K]
    uint16_t* out;              // GATE_UP: Hm [rows, N]; DOWN: D [rows, N]
    const int* perm;            // [rows] flat (token, slot) index of permuted row r
    const int* topk_idx;        // [T*topk]
    int rows, topk, N, K;       // N, K of one expert matrix
};

enum { kMoeGateUp = 0, kMoeDown = 1 };

template <int FMT, int MODE, int WARPS>
__global__ void __launch_bounds__(WARPS * 32, 768 / (WARPS * 32))
moe_gemv_kernel(const MoeGemvParams p)
{
    extern __shared__ uint4 smem[];
    uint4* xs = smem;
    uint4* zs = smem + p.K / 8;
    float* red = reinterpret_cast<float*>(smem + p.K / 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int TB = Fmt<FMT>::tile_bytes;
    constexpr int XV = Fmt<FMT>::tile_k / 8;
    constexpr int STEP = kUnroll * WARPS;
    constexpr int OUT_PER_UNIT = MODE == kMoeGateUp ? 32 : 64;
    const int tpr = p.K / Fmt<FMT>::tile_k;
    const int units_per_row = p.N / OUT_PER_UNIT;
    const int units = p.rows * units_per_row;
    const size_t group_bytes = (size_t)tpr * TB;

    pdl_launch_dependents();
    pdl_wait();                                                 // routing result and activations are written upstream
    for (int i = threadIdx.x; i < p.K / 8; i += WARPS * 32) zs[i] = make_uint4(0u, 0u, 0u, 0u);
    const uint4* xb = ((lane >> 2) == (lane & 3)) ? xs : zs;
    Q4Consts kc;
    kc.init();

    int cur_row = -1;
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
        const int r = u / units_per_row, j = u - r * units_per_row;
        const int flat = p.perm[r];
        const int e = p.topk_idx[flat];
        if (r != cur_row) {                                     // stage this row's activation vector
            __syncthreads();
            const uint16_t* xr = MODE == kMoeGateUp ? p.x + (size_t)(flat / p.topk) * p.K : p.x + (size_t)r * p.K;
            for (int i = threadIdx.x; i < p.K / 8; i += WARPS * 32) xs[i] = reinterpret_cast<const uint4*>(xr)[i];
            __syncthreads();
            cur_row = r;
        }
        const uint8_t *tiles_p, *tiles_q;
        if (MODE == kMoeGateUp) {
            tiles_p = p.w0 + (size_t)e * p.expert_stride + (size_t)j * group_bytes + 32 * lane;
            tiles_q = p.w1 + (size_t)e * p.expert_stride + (size_t)j * group_bytes + 32 * lane;
        } else {
            tiles_p = p.w0 + (size_t)e * p.expert_stride + (size_t)(2 * j) * group_bytes + 32 * lane;
            tiles_q = tiles_p + group_bytes;
        }
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int t = warp; t < tpr; t += STEP) {
            TileRegs<FMT> rg;
#pragma unroll
            for (int q = 0; q < kUnroll; ++q) {
                const int tt = t + q * WARPS;
                if (tt < tpr) {
                    const uint8_t* tp = tiles_p + (size_t)tt * TB;
                    const uint8_t* tq = tiles_q + (size_t)tt * TB;
                    rg.cp[q] = ld_stream_256(tp);
                    rg.cq[q] = ld_stream_256(tq);
                    rg.sp[q] = load_scales<FMT>(tp - 32 * lane, lane);
                    rg.sq[q] = load_scales<FMT>(tq - 32 * lane, lane);
                }
            }
#pragma unroll
            for (int q = 0; q < kUnroll; ++q) {
                const int tt = t + q * WARPS;
                if (tt < tpr) {
                    if constexpr (FMT == QMM_Q4)
                        tile_pair_mma_q4(rg.cp[q], rg.cq[q], rg.sp[q], rg.sq[q], xb + tt * XV, acc, kc);
                    else
                        tile_pair_mma_q8(rg.cp[q], rg.cq[q], rg.sp[q], rg.sq[q], xb + tt * XV, acc);
                }
            }
        }
        if ((lane & 3) < 2) {
            const int row = (lane & ~3) + 2 * (lane & 1);
            float* w = red + warp * 64;
            w[row] = acc[0];
            w[row + 1] = acc[1];
            w[32 + row] = acc[2];
            w[32 + row + 1] = acc[3];
        }
        __syncthreads();
        if (MODE == kMoeGateUp) {
            if (threadIdx.x < 32) {                             // red[.. 0..31] = G, red[.. 32..63] = U
                float g = red[threadIdx.x], up = red[32 + threadIdx.x];
#pragma unroll
                for (int w = 1; w < WARPS; ++w) {
                    g += red[w * 64 + threadIdx.x];
                    up += red[w * 64 + 32 + threadIdx.x];
                }
                const float h = (g / (1.0f + expf(-g))) * up;
                p.out[(size_t)r * p.N + j * 32 + threadIdx.x] = __half_as_ushort(__float2half_rn(h));
            }
        } else {
            if (threadIdx.x < 64) {
                float sum = red[threadIdx.x];
#pragma unroll
                for (int w = 1; w < WARPS; ++w) sum += red[w * 64 + threadIdx.x];
                p.out[(size_t)r * p.N + j * 64 + threadIdx.x] = __half_as_ushort(__float2half_rn(sum));
            }
        }
        __syncthreads();
    }
}

// ------------------------------------------- MoE decode layer in two launches
//
// Decode-sized layers (T * topk <= 32 rows, topk <= 8).  Four dependent launches of ~5 us each
// (route, gate/up, down, combine) around ~3 us of weight traffic is what a layer per-launch costs;
// the paper's decode argument is exactly that such dispatch cost, not bytes, dominates short kernels
// (Sec. 3.3).  Here the layer is two launches:
//   A: every block routes all T tokens itself (T * E logits: a few KB, ~1 us) instead of waiting for a
//      routing kernel, then runs its gate/up units with the SiLU*mul epilogue; block 0 also writes the
//      routing results (indices, weights, permutation, offsets) for the caller.
//   B: a thread-block cluster per (token, 64 output columns); cluster rank j takes the token's j-th
//      expert, multiplies the expert's 64 down rows with Hm[row(t, j)], rounds to fp16 (the library's
//      D), and the cluster's first block adds p_j * D_j in slot order through distributed shared
//      memory and writes `out` -- D never leaves the SMs and no combine kernel runs.  B routes again
//      from the logits (an input that is complete before A started), so its blocks know their expert
//      and prefetch its weights *before* they wait for A's Hm.
struct MoeSmallParams {
    const float* logits;        // [T, E]
    const uint16_t* X;          // [T, H]
    const uint8_t *w_gate, *w_up, *w_down;
    int64_t gu_stride, dn_stride;   // bytes between experts
    uint16_t* hbuf;             // [T*topk, I] permuted row order (workspace or dbg_H)
    uint16_t* dbg_D;            // [T*topk, H] optional export of D
    uint16_t* out;              // [T, H]
    int T, E, topk, H, I;
    int* idx_ws;                // workspace copies of the routing result (read by nothing downstream, kept for qmm_moe_route parity)
    float* w_ws;
    int *perm_ws, *inv_ws, *offsets_ws;
    int* idx_user;              // optional exports
    float* w_user;
    int *perm_user, *offsets_user;
    long long* trace;           // -DQMM_MOE_TRACE=1 builds: %globaltimer samples of block 0 of each launch; else unused
};

// Time stamps of the two launches' first blocks (tuning builds only; the shipped kernels carry none).
#ifndef QMM_MOE_TRACE
#define QMM_MOE_TRACE 0
#endif
#if QMM_MOE_TRACE
#define QMM_MOE_STAMP(i)                                                        \
    if (blockIdx.x == 0 && threadIdx.x == 0 && p.trace != nullptr) {            \
        long long t_;                                                           \
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_));                  \
        p.trace[i] = t_;                                                        \
    }
#else
#define QMM_MOE_STAMP(i)
#endif

// Routing + stable permutation of all T * topk <= 32 (token, slot) pairs by the whole block.
// s_e / s_w: expert and weight of flat pair t * topk + j; s_perm[r] = flat pair of permuted row r;
// s_inv[flat] = r.  Same selection rule and arithmetic as route_kernel, so every block (and the
// separate routing kernels) get the same bits.
template <int MAX_PER_LANE, int WARPS>
__device__ __forceinline__ void route_all(const float* __restrict__ logits, int T, int E, int topk,
                                          int* s_e, float* s_w, int* s_perm, int* s_inv)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int total = T * topk;
    for (int t = warp; t < T; t += WARPS) {
        int sel_idx;
        float w;
        route_token<MAX_PER_LANE>(logits + (size_t)t * E, E, topk, lane, sel_idx, w);
        if (lane < topk) {
            s_e[t * topk + lane] = sel_idx;
            s_w[t * topk + lane] = w;
        }
    }
    __syncthreads();
    if ((int)threadIdx.x < total) {                          // rank of this pair in the (expert, flat index) order
        const int mine = s_e[threadIdx.x];
        int r = 0;
        for (int j = 0; j < total; ++j) {
            const int other = s_e[j];
            r += (other < mine || (other == mine && j < (int)threadIdx.x)) ? 1 : 0;
        }
        s_perm[r] = threadIdx.x;
        s_inv[threadIdx.x] = r;
    }
    __syncthreads();
}

// Four tile pairs in flight per warp (twice the GEMV's): a decode unit is one short stream (gate and up
// rows of 32 outputs), and every round of loads it needs is a full memory latency on the layer's
// critical path -- K = 2048 in the 4-bit format is one round this way.
constexpr int kMoeSmallUnroll = 4;

template <int FMT, int MAX_PER_LANE, int WARPS>
__global__ void __launch_bounds__(WARPS * 32, 512 / (WARPS * 32))
moe_small_gate_up_kernel(const MoeSmallParams p)
{
    extern __shared__ uint4 smem[];
    uint4* xs = smem;
    uint4* zs = smem + p.H / 8;
    float* red = reinterpret_cast<float*>(smem + p.H / 4);
    __shared__ int s_e[32], s_perm[32], s_inv[32];
    __shared__ float s_w[32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int TB = Fmt<FMT>::tile_bytes;
    constexpr int XV = Fmt<FMT>::tile_k / 8;
    constexpr int UNR = kMoeSmallUnroll;
    constexpr int STEP = UNR * WARPS;
    const int K = p.H, N = p.I;
    const int tpr = K / Fmt<FMT>::tile_k;
    const int units_per_row = N / 32;
    const int total = p.T * p.topk;
    const int units = total * units_per_row;
    const size_t group_bytes = (size_t)tpr * TB;

    QMM_MOE_STAMP(0)
    pdl_wait();                                                 // logits and activations come from upstream
    pdl_launch_dependents();
    QMM_MOE_STAMP(1)
    route_all<MAX_PER_LANE, WARPS>(p.logits, p.T, p.E, p.topk, s_e, s_w, s_perm, s_inv);
    QMM_MOE_STAMP(2)
    if (blockIdx.x == 0) {                                      // the routing result, for the caller and the workspace
        if ((int)threadIdx.x < total) {
            const int i = threadIdx.x;
            p.idx_ws[i] = s_e[i];
            p.w_ws[i] = s_w[i];
            p.perm_ws[i] = s_perm[i];
            p.inv_ws[i] = s_inv[i];
            if (p.idx_user) p.idx_user[i] = s_e[i];
            if (p.w_user) p.w_user[i] = s_w[i];
            if (p.perm_user) p.perm_user[i] = s_perm[i];
        }
        for (int e = threadIdx.x; e <= p.E; e += WARPS * 32) {  // rows of the experts before e
            int c = 0;
            for (int j = 0; j < total; ++j) c += s_e[j] < e ? 1 : 0;
            p.offsets_ws[e] = c;
            if (p.offsets_user) p.offsets_user[e] = c;
        }
    }
    for (int i = threadIdx.x; i < K / 8; i += WARPS * 32) zs[i] = make_uint4(0u, 0u, 0u, 0u);
    const uint4* xb = ((lane >> 2) == (lane & 3)) ? xs : zs;
    Q4Consts kc;
    kc.init();

    int cur_row = -1;
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
        const int r = u / units_per_row, j = u - r * units_per_row;
        const int flat = s_perm[r];
        const int e = s_e[flat];
        const uint8_t* tiles_p = p.w_gate + (size_t)e * p.gu_stride + (size_t)j * group_bytes + 32 * lane;
        const uint8_t* tiles_q = p.w_up + (size_t)e * p.gu_stride + (size_t)j * group_bytes + 32 * lane;
        struct {
            u32x8 cp[UNR], cq[UNR];
            typename ScaleRegs<FMT>::type sp[UNR], sq[UNR];
        } rg;
        auto load_group = [&](int t) {
#pragma unroll
            for (int q = 0; q < UNR; ++q) {
                const int tt = t + q * WARPS;
                if (tt < tpr) {
                    const uint8_t* tp = tiles_p + (size_t)tt * TB;
                    const uint8_t* tq = tiles_q + (size_t)tt * TB;
                    rg.cp[q] = ld_stream_256(tp);
                    rg.cq[q] = ld_stream_256(tq);
                    rg.sp[q] = load_scales<FMT>(tp - 32 * lane, lane);
                    rg.sq[q] = load_scales<FMT>(tq - 32 * lane, lane);
                }
            }
        };
        load_group(warp);                                       // weights fly while the activation row is staged
        if (r != cur_row) {
            __syncthreads();
            const uint16_t* xr = p.X + (size_t)(flat / p.topk) * K;
            for (int i = threadIdx.x; i < K / 8; i += WARPS * 32) xs[i] = reinterpret_cast<const uint4*>(xr)[i];
            __syncthreads();
            cur_row = r;
        }
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int t = warp; t < tpr; t += STEP) {
#pragma unroll
            for (int q = 0; q < UNR; ++q) {
                const int tt = t + q * WARPS;
                if (tt < tpr) {
                    if constexpr (FMT == QMM_Q4)
                        tile_pair_mma_q4(rg.cp[q], rg.cq[q], rg.sp[q], rg.sq[q], xb + tt * XV, acc, kc);
                    else
                        tile_pair_mma_q8(rg.cp[q], rg.cq[q], rg.sp[q], rg.sq[q], xb + tt * XV, acc);
                }
            }
            if (t + STEP < tpr) load_group(t + STEP);
        }
        QMM_MOE_STAMP(3)
        if ((lane & 3) < 2) {
            const int row = (lane & ~3) + 2 * (lane & 1);
            float* w = red + warp * 64;
            w[row] = acc[0];
            w[row + 1] = acc[1];
            w[32 + row] = acc[2];
            w[32 + row + 1] = acc[3];
        }
        __syncthreads();
        if (threadIdx.x < 32) {                                 // red[.. 0..31] = G, red[.. 32..63] = U
            float g = red[threadIdx.x], up = red[32 + threadIdx.x];
#pragma unroll
            for (int w = 1; w < WARPS; ++w) {
                g += red[w * 64 + threadIdx.x];
                up += red[w * 64 + 32 + threadIdx.x];
            }
            const float h = (g / (1.0f + expf(-g))) * up;
            p.hbuf[(size_t)r * N + j * 32 + threadIdx.x] = __half_as_ushort(__float2half_rn(h));
        }
        __syncthreads();
        QMM_MOE_STAMP(4)
    }
}

// Launch B (see above).  gridDim.x = T * (H / 64) * topk, cluster = topk blocks.
template <int FMT, int MAX_PER_LANE, int WARPS>
__global__ void __launch_bounds__(WARPS * 32, 768 / (WARPS * 32))
moe_small_down_combine_kernel(const MoeSmallParams p)
{
    extern __shared__ uint4 smem[];
    uint4* xs = smem;
    uint4* zs = smem + p.I / 8;
    float* red = reinterpret_cast<float*>(smem + p.I / 4);
    float* cred = red + WARPS * 64;                             // [kMaxClusterSplits][64] in the cluster's first block
    __shared__ int s_e[32], s_perm[32], s_inv[32];
    __shared__ float s_w[32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int TB = Fmt<FMT>::tile_bytes;
    constexpr int XV = Fmt<FMT>::tile_k / 8;
    constexpr int STEP = kUnroll * WARPS;
    const int K = p.I, N = p.H;
    const int tpr = K / Fmt<FMT>::tile_k;
    const size_t group_bytes = (size_t)tpr * TB;
    // every block of the cluster has started once this barrier phase completes (awaited before the
    // first store into the first block's shared memory)
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    const int slot = blockIdx.x % p.topk;                       // rank in the cluster = the token's slot j
    const int cu = blockIdx.x / p.topk;
    const int col_groups = N / 64;
    const int t = cu / col_groups, g = cu - t * col_groups;     // token, group of 64 output columns

    QMM_MOE_STAMP(8)
    // the logits are an input of the layer: complete before launch A started, so they can be read now
    route_all<MAX_PER_LANE, WARPS>(p.logits, p.T, p.E, p.topk, s_e, s_w, s_perm, s_inv);
    QMM_MOE_STAMP(9)
    const int flat = t * p.topk + slot;
    const int e = s_e[flat];
    const int r = s_inv[flat];                                  // permuted row of (t, slot)
    const uint8_t* tiles_p = p.w_down + (size_t)e * p.dn_stride + (size_t)(2 * g) * group_bytes + 32 * lane;
    const uint8_t* tiles_q = tiles_p + group_bytes;
    TileRegs<FMT> rg;
    auto load_group = [&](int t0) {
#pragma unroll
        for (int q = 0; q < kUnroll; ++q) {
            const int tt = t0 + q * WARPS;
            if (tt < tpr) {
                const uint8_t* tp = tiles_p + (size_t)tt * TB;
                const uint8_t* tq = tiles_q + (size_t)tt * TB;
                rg.cp[q] = ld_stream_256(tp);
                rg.cq[q] = ld_stream_256(tq);
                rg.sp[q] = load_scales<FMT>(tp - 32 * lane, lane);
                rg.sq[q] = load_scales<FMT>(tq - 32 * lane, lane);
            }
        }
    };
    load_group(warp);                                           // the expert's weights, ahead of the wait for Hm
    for (int i = threadIdx.x; i < K / 8; i += WARPS * 32) zs[i] = make_uint4(0u, 0u, 0u, 0u);

    pdl_launch_dependents();
    pdl_wait();                                                 // Hm is written by launch A
    QMM_MOE_STAMP(10)
    {
        const uint16_t* xr = p.hbuf + (size_t)r * K;
        for (int i = threadIdx.x; i < K / 8; i += WARPS * 32) xs[i] = __ldcg(reinterpret_cast<const uint4*>(xr) + i);
    }
    __syncthreads();
    const uint4* xb = ((lane >> 2) == (lane & 3)) ? xs : zs;
    Q4Consts kc;
    kc.init();
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int t0 = warp; t0 < tpr; t0 += STEP) {
#pragma unroll
        for (int q = 0; q < kUnroll; ++q) {
            const int tt = t0 + q * WARPS;
            if (tt < tpr) {
                if constexpr (FMT == QMM_Q4)
                    tile_pair_mma_q4(rg.cp[q], rg.cq[q], rg.sp[q], rg.sq[q], xb + tt * XV, acc, kc);
                else
                    tile_pair_mma_q8(rg.cp[q], rg.cq[q], rg.sp[q], rg.sq[q], xb + tt * XV, acc);
            }
        }
        if (t0 + STEP < tpr) load_group(t0 + STEP);
    }
    if ((lane & 3) < 2) {
        const int row = (lane & ~3) + 2 * (lane & 1);
        float* w = red + warp * 64;
        w[row] = acc[0];
        w[row + 1] = acc[1];
        w[32 + row] = acc[2];
        w[32 + row + 1] = acc[3];
    }
    __syncthreads();
    QMM_MOE_STAMP(11)
    asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
    if (threadIdx.x < 64) {
        float sum = red[threadIdx.x];
#pragma unroll
        for (int w = 1; w < WARPS; ++w) sum += red[w * 64 + threadIdx.x];
        const __half d = __float2half_rn(sum);                  // D is an fp16 tensor of the layer's definition
        if (p.dbg_D) p.dbg_D[(size_t)r * N + g * 64 + threadIdx.x] = __half_as_ushort(d);
        st_cluster_rank0(cred + slot * 64 + threadIdx.x, __half2float(d));
    }
    cluster_sync();
    QMM_MOE_STAMP(12)
    if (slot == 0 && threadIdx.x < 64) {                        // out = fp16(sum_j p_j * D_j), j ascending, as combine_kernel
        float o = 0.f;
        for (int j = 0; j < p.topk; ++j) o = fmaf(s_w[t * p.topk + j], cred[j * 64 + threadIdx.x], o);
        p.out[(size_t)t * N + g * 64 + threadIdx.x] = __half_as_ushort(__float2half_rn(o));
    }
}

// Second stage of split-K: y[n] = fp16(sum_s partial[s][n]), s ascending.
__global__ void gemv_reduce_kernel(const float* __restrict__ partial, uint16_t* __restrict__ y, int N, int splits)
{
    pdl_launch_dependents();
    pdl_wait();
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N) return;
    float sum = partial[n];
    for (int s = 1; s < splits; ++s) sum += partial[(size_t)s * N + n];
    y[n] = __half_as_ushort(__float2half_rn(sum));
}

// ------------------------------------------------------------------ host

struct GemvPlan {
    int warps;    // 8 or 16
    int splits;   // K splits across thread blocks
    int grid;
};

// Shape -> launch geometry.  The aim is >= ~2 resident blocks' worth of loads
// on every SM: prefer more warps per block, and split K across blocks only
// when the row groups alone cannot cover the SMs.
GemvPlan gemv_plan(int fmt, int64_t N, int64_t K, bool cluster)
{
    GemvPlan p;
    const int tpr = (int)(K / tile_k_of(fmt));
    const int groups = (int)(N / (2 * kRowsPerGroup));       // items are pairs of row groups
    int warps = 16;                                           // <= 512 threads: two generations of blocks fit on an SM
    while (warps > 8 && warps > tpr) warps >>= 1;
    // large problems: fewer warps per block so that several blocks share an SM
    if ((int64_t)groups * tpr >= (int64_t)kNumSMs * 64 * 4 && warps > 8) warps = 8;
    else if ((int64_t)groups * tpr >= (int64_t)kNumSMs * 64 && warps > 16) warps = 16;
    int splits = 1;
    const int max_splits = cluster ? kPlanClusterSplits : 16;
    while (groups * splits < kNumSMs && tpr / (splits * 2) >= warps && (tpr % (splits * 2)) == 0 && splits < max_splits)
        splits *= 2;
    if (g_knobs.gemv_warps && tpr % g_knobs.gemv_splits == 0) {   // forced by qmm_debug_config("gemv_force", "warps,splits")
        warps = g_knobs.gemv_warps;
        splits = g_knobs.gemv_splits;
    }
    p.warps = warps;
    p.splits = splits;
    const int items = groups * splits;
    const int per_sm = 768 / (warps * 32);
    p.grid = items < kNumSMs * per_sm ? items : kNumSMs * per_sm;
    return p;
}

// Workspace of the K split.  The cluster form (up to kMaxClusterSplits blocks per item, sums added
// through distributed shared memory) needs none; the two-kernel form holds fp32 partial sums [splits][N].
size_t gemv_workspace_bytes(int fmt, int64_t N, int64_t K, bool allow_cluster)
{
    if (g_knobs.gemv_no_cluster) allow_cluster = false;
    const GemvPlan p = gemv_plan(fmt, N, K, allow_cluster);
    if (p.splits <= 1 || (allow_cluster && p.splits <= kMaxClusterSplits)) return 0;
    return (size_t)p.splits * (size_t)N * sizeof(float);
}

template <typename... Args>
static cudaError_t launch_pdl(void (*kernel)(Args...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

template <int FMT, int WARPS>
static qmm_status launch_gemv_t(const GemvPlan& p, const void* packed, int64_t N, int64_t K,
                                const uint16_t* x, uint16_t* y, float* partial, bool allow_cluster, cudaStream_t st)
{
    // K split over up to 8 blocks: the blocks of an item form a cluster and add their sums through
    // distributed shared memory; more splits (or a caller that brings its own scratch): partial sums
    // in memory and a second kernel
    const bool cluster = allow_cluster && p.splits > 1 && p.splits <= kMaxClusterSplits;
    const size_t smem = (size_t)K * 4 + (size_t)WARPS * 64 * sizeof(float) + (cluster ? 2 * kMaxClusterSplits * 64 * sizeof(float) : 0);
    auto kern = gemv_kernel<FMT, WARPS>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemv shared memory size");
    }
    const int tpr = (int)(K / Fmt<FMT>::tile_k);
    const int items = (int)(N / (2 * kRowsPerGroup)) * p.splits;
    if (cluster) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(p.grid / p.splits * p.splits));      // whole clusters
        cfg.blockDim = dim3(WARPS * 32);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)p.splits;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        return check_cuda(cudaLaunchKernelEx(&cfg, kern, (const uint8_t*)packed, x, y, (float*)nullptr, (int)N, (int)K, tpr, p.splits,
                                             items, (const uint8_t*)nullptr, (int64_t)0, (int64_t)0),
                          "qmm_gemv cluster launch");
    }
    cudaError_t e = launch_pdl(kern, dim3(p.grid), dim3(WARPS * 32), smem, st,
                               (const uint8_t*)packed, x, y, partial, (int)N, (int)K, tpr, p.splits, items, (const uint8_t*)nullptr, (int64_t)0, (int64_t)0);
    if (e != cudaSuccess) return check_cuda(e, "qmm_gemv launch");
    if (p.splits > 1) {
        e = launch_pdl(gemv_reduce_kernel, dim3((unsigned)((N + 255) / 256)), dim3(256), 0, st,
                       (const float*)partial, y, (int)N, p.splits);
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemv reduce launch");
    }
    return QMM_OK;
}

// h = fp16(silu(W_gate x) * (W_up x)): gemv_kernel with (gate group, up group) pairs, one item per 32 outputs.
qmm_status launch_gemv_gate_up(int fmt, const void* packed_gate, const void* packed_up, int64_t N, int64_t K,
                               const uint16_t* x, uint16_t* h, cudaStream_t st)
{
    constexpr int WARPS = 8;
    const size_t smem = (size_t)K * 4 + (size_t)WARPS * 64 * sizeof(float);
    const int tpr = (int)(K / tile_k_of(fmt));
    const int items = (int)(N / kRowsPerGroup);
    const int grid = items < 3 * kNumSMs ? items : 3 * kNumSMs;
    cudaError_t e = cudaSuccess;
    if (fmt == QMM_Q4) {
        auto kern = gemv_kernel<QMM_Q4, WARPS, true>;
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess)
            e = launch_pdl(kern, dim3(grid), dim3(WARPS * 32), smem, st, (const uint8_t*)packed_gate, x, h, (float*)nullptr, (int)N,
                           (int)K, tpr, 1, items, (const uint8_t*)packed_up, (int64_t)0, (int64_t)0);
    } else {
        auto kern = gemv_kernel<QMM_Q8, WARPS, true>;
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e == cudaSuccess)
            e = launch_pdl(kern, dim3(grid), dim3(WARPS * 32), smem, st, (const uint8_t*)packed_gate, x, h, (float*)nullptr, (int)N,
                           (int)K, tpr, 1, items, (const uint8_t*)packed_up, (int64_t)0, (int64_t)0);
    }
    return check_cuda(e, "qmm_gemv_gate_up launch");
}

// Expert products of the MoE layer for a handful of rows (decode): see moe_gemv_kernel.
qmm_status launch_moe_gemv(int fmt, bool gate_up, const void* w0, const void* w1, int64_t expert_stride,
                           const uint16_t* x, uint16_t* out, const int* perm, const int* topk_idx,
                           int rows, int topk, int N, int K, cudaStream_t st)
{
    constexpr int WARPS = 8;
    MoeGemvParams p;
    p.w0 = (const uint8_t*)w0;
    p.w1 = (const uint8_t*)w1;
    p.expert_stride = expert_stride;
    p.x = x;
    p.out = out;
    p.perm = perm;
    p.topk_idx = topk_idx;
    p.rows = rows;
    p.topk = topk;
    p.N = N;
    p.K = K;
    const size_t smem = (size_t)K * 4 + (size_t)WARPS * 64 * sizeof(float);
    const int units = rows * (N / (gate_up ? 32 : 64));
    const int grid = units < kNumSMs * 3 ? units : kNumSMs * 3;
    cudaError_t e = cudaSuccess;
#define QMM_MOE_GEMV(F, M)                                                                                        \
    {                                                                                                             \
        auto kern = moe_gemv_kernel<F, M, WARPS>;                                                                 \
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
        if (e == cudaSuccess) e = launch_pdl(kern, dim3(grid), dim3(WARPS * 32), smem, st, p);                    \
    }
    if (fmt == QMM_Q4 && gate_up) QMM_MOE_GEMV(QMM_Q4, kMoeGateUp)
    else if (fmt == QMM_Q4) QMM_MOE_GEMV(QMM_Q4, kMoeDown)
    else if (gate_up) QMM_MOE_GEMV(QMM_Q8, kMoeGateUp)
    else QMM_MOE_GEMV(QMM_Q8, kMoeDown)
#undef QMM_MOE_GEMV
    return check_cuda(e, "qmm_moe decode GEMV launch");
}

// Decode-sized MoE layer in two launches (see moe_small_gate_up_kernel).

template <int FMT, int MPL>
static qmm_status launch_moe_small_t(const MoeSmallParams& p, bool route_only, cudaStream_t st)
{
    constexpr int WARPS = 8;
    const int total = p.T * p.topk;
    {
        auto kern = moe_small_gate_up_kernel<FMT, MPL, WARPS>;
        const size_t smem = (size_t)p.H * 4 + (size_t)WARPS * 64 * sizeof(float);
        cudaError_t e = cudaSuccess;
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return check_cuda(e, "qmm_moe decode gate/up shared memory size");
        const int units = route_only ? 0 : total * (p.I / 32);
        int grid = units < kNumSMs * 2 ? units : kNumSMs * 2;
        if (grid < 1) grid = 1;                                 // block 0 always exports the routing result
        MoeSmallParams q = p;
        if (route_only) q.I = 0;                                // no units: routing only
        e = launch_pdl(kern, dim3(grid), dim3(WARPS * 32), smem, st, q);
        if (e != cudaSuccess) return check_cuda(e, "qmm_moe decode gate/up launch");
    }
    if (route_only) return QMM_OK;
    {
        auto kern = moe_small_down_combine_kernel<FMT, MPL, WARPS>;
        const size_t smem = (size_t)p.I * 4 + (size_t)WARPS * 64 * sizeof(float) + kMaxClusterSplits * 64 * sizeof(float);
        cudaError_t e = cudaSuccess;
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return check_cuda(e, "qmm_moe decode down shared memory size");
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(p.T * (p.H / 64) * p.topk));
        cfg.blockDim = dim3(WARPS * 32);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)p.topk;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        e = cudaLaunchKernelEx(&cfg, kern, p);
        if (e != cudaSuccess) return check_cuda(e, "qmm_moe decode down + combine launch");
    }
    return QMM_OK;
}

// Limits of the two-launch form: the pairs fit one warp's ranking pass, the experts of a token fit a
// portable cluster, a row of X / Hm fits the shared-memory staging.
// It is taken while the gate/up units fit the SMs in one wave (two blocks of 128 registers per thread
// per SM): beyond that the four-launch form, whose GEMV kernels keep three lighter blocks per SM, was
// measured equal (T = 2 at the 128-expert, top-8 layer: 27.5 us both) or faster (T = 4: 38 against 42 us).
bool moe_small_supported(int T, int topk, int H, int I)
{
    return T * topk <= 32 && topk <= kMaxClusterSplits && H <= 32768 && I <= 32768 && H % 64 == 0 && I % 32 == 0 &&
           (int64_t)T * topk * (I / 32) <= 2 * kNumSMs;
}

qmm_status launch_moe_small(int fmt, const MoeSmallHost& h, bool route_only, cudaStream_t st)
{
    MoeSmallParams p;
    p.logits = h.logits; p.X = h.X;
    p.w_gate = (const uint8_t*)h.w_gate; p.w_up = (const uint8_t*)h.w_up; p.w_down = (const uint8_t*)h.w_down;
    p.gu_stride = h.gu_stride; p.dn_stride = h.dn_stride;
    p.hbuf = h.hbuf; p.dbg_D = h.dbg_D; p.out = h.out;
    p.T = h.T; p.E = h.E; p.topk = h.topk; p.H = h.H; p.I = h.I;
    p.idx_ws = h.idx_ws; p.w_ws = h.w_ws; p.perm_ws = h.perm_ws; p.inv_ws = h.inv_ws; p.offsets_ws = h.offsets_ws;
    p.idx_user = h.idx_user; p.w_user = h.w_user; p.perm_user = h.perm_user; p.offsets_user = h.offsets_user;
    p.trace = h.trace;
    const bool narrow = (h.E + 31) / 32 <= 4;
    if (fmt == QMM_Q4) return narrow ? launch_moe_small_t<QMM_Q4, 4>(p, route_only, st) : launch_moe_small_t<QMM_Q4, 32>(p, route_only, st);
    return narrow ? launch_moe_small_t<QMM_Q8, 4>(p, route_only, st) : launch_moe_small_t<QMM_Q8, 32>(p, route_only, st);
}

// Host side of qmm_gemv_batch: up to kMaxBatch problems per launch.
qmm_status launch_gemv_batch(int fmt, const qmm_gemv_problem* probs, int count, cudaStream_t st, bool out_f32)
{
    for (int first = 0; first < count; first += kMaxBatch) {
        const int n = count - first < kMaxBatch ? count - first : kMaxBatch;
        BatchParams bp = {};
        bp.count = n;
        bp.out_f32 = out_f32 ? 1 : 0;
        int cost = 0, max_k = 0;
        for (int i = 0; i < n; ++i) {
            const qmm_gemv_problem& q = probs[first + i];
            BatchProblem& b = bp.p[i];
            b.packed = (const uint8_t*)q.packed;
            b.x = q.x_fp16;
            b.y = q.y_fp16;
            b.K = (int)q.K;
            b.tpr = (int)(q.K / tile_k_of(fmt));
            b.pairs = (int)(q.N / (2 * kRowsPerGroup));
            b.cost_begin = cost;
            if ((long long)cost + (long long)b.pairs * b.tpr > 0x7FFFFFFFLL)
                return fail(QMM_ERR_UNSUPPORTED, "qmm_gemv_batch: batch too large for one launch");
            cost += b.pairs * b.tpr;
            if (b.K > max_k) max_k = b.K;
        }
        bp.total_cost = cost;
        bp.max_k = max_k;
        constexpr int WARPS = 8;
        const size_t smem = (size_t)max_k * 4 + (size_t)WARPS * 64 * sizeof(float);
        const int units = cost / (max_k / tile_k_of(fmt)) + 1;
        int grid = kNumSMs * (QMM_BATCH_THREADS_PER_SM / (WARPS * 32));
        if (units < grid) grid = units;
        cudaError_t e;
#define QMM_BATCH_CASE(F)                                                                                                          \
    {                                                                                                                              \
        auto kern = gemv_batch_kernel<F, WARPS>;                                                                                   \
        if (smem > 48 * 1024 && (e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) \
            return check_cuda(e, "qmm_gemv_batch shared memory size");                                                             \
        e = launch_pdl(kern, dim3(grid), dim3(WARPS * 32), smem, st, bp);                                                          \
    }
        if (fmt == QMM_Q4) QMM_BATCH_CASE(QMM_Q4)
        else if (fmt == QMM_Q5) QMM_BATCH_CASE(QMM_Q5)
        else if (fmt == QMM_Q6) QMM_BATCH_CASE(QMM_Q6)
        else QMM_BATCH_CASE(QMM_Q8)
#undef QMM_BATCH_CASE
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemv_batch launch");
    }
    return QMM_OK;
}

// qmm_gemm for two tokens: gemv_kernel's TWO form.  Returns QMM_ERR_UNSUPPORTED without touching the error text
// when the shape needs the workspace form of the K split or more shared memory than a block has; the caller
// then takes its other kernel.
template <int FMT, int WARPS>
static qmm_status launch_gemv_two_t(const GemvPlan& p, const void* packed, int64_t N, int64_t K, const uint16_t* X, int64_t ldx,
                                    uint16_t* Y, int64_t ldy, cudaStream_t st)
{
    const bool cluster = p.splits > 1;
    const size_t smem = (size_t)K * 6 + (size_t)WARPS * 128 * sizeof(float) + (cluster ? 2 * kMaxClusterSplits * 128 * sizeof(float) : 0);
    if (smem > 227 * 1024) return QMM_ERR_UNSUPPORTED;
    auto kern = gemv_kernel<FMT, WARPS, false, true>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemm two-token kernel shared memory size");
    }
    const int tpr = (int)(K / Fmt<FMT>::tile_k);
    const int items = (int)(N / (2 * kRowsPerGroup)) * p.splits;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(cluster ? p.grid / p.splits * p.splits : p.grid));
    cfg.blockDim = dim3(WARPS * 32);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)p.splits;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cluster ? 2 : 1;
    return check_cuda(cudaLaunchKernelEx(&cfg, kern, (const uint8_t*)packed, X, Y, (float*)nullptr, (int)N, (int)K, tpr, p.splits, items,
                                         (const uint8_t*)nullptr, ldx, ldy),
                      "qmm_gemm two-token kernel launch");
}

bool gemv_two_supported(int fmt, int64_t N, int64_t K)
{
    if (K > 32768 || g_knobs.gemv_no_cluster) return false;
    const GemvPlan p = gemv_plan(fmt, N, K, true);
    return p.splits <= kMaxClusterSplits;
}

qmm_status launch_gemv_two(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* X, int64_t ldx, uint16_t* Y,
                           int64_t ldy, cudaStream_t st)
{
    const GemvPlan p = gemv_plan(fmt, N, K, true);
#define QMM_GEMV2_CASE(F, W) \
    if (fmt == F && p.warps == W) return launch_gemv_two_t<F, W>(p, packed, N, K, X, ldx, Y, ldy, st);
    QMM_GEMV2_CASE(QMM_Q4, 8)
    QMM_GEMV2_CASE(QMM_Q4, 16)
    QMM_GEMV2_CASE(QMM_Q8, 8)
    QMM_GEMV2_CASE(QMM_Q8, 16)
    QMM_GEMV2_CASE(QMM_Q5, 8)
    QMM_GEMV2_CASE(QMM_Q5, 16)
    QMM_GEMV2_CASE(QMM_Q6, 8)
    QMM_GEMV2_CASE(QMM_Q6, 16)
#undef QMM_GEMV2_CASE
    return QMM_ERR_UNSUPPORTED;
}

// qmm_gemm_batch for two tokens: the batched kernel's TWO form (both tokens at the cost of one).
qmm_status launch_gemv_batch_two(int fmt, const qmm_gemm_problem* probs, int count, cudaStream_t st)
{
    for (int first = 0; first < count; first += kMaxBatch) {
        const int n = count - first < kMaxBatch ? count - first : kMaxBatch;
        BatchParams bp = {};
        bp.count = n;
        int cost = 0, max_k = 0;
        for (int i = 0; i < n; ++i) {
            const qmm_gemm_problem& q = probs[first + i];
            BatchProblem& b = bp.p[i];
            b.packed = (const uint8_t*)q.packed;
            b.x = q.X_fp16;
            b.x2 = q.X_fp16 + q.ldx;
            b.y = q.Y_fp16;
            b.y2 = q.Y_fp16 + q.ldy;
            b.K = (int)q.K;
            b.tpr = (int)(q.K / tile_k_of(fmt));
            b.pairs = (int)(q.N / (2 * kRowsPerGroup));
            b.cost_begin = cost;
            if ((long long)cost + (long long)b.pairs * b.tpr > 0x7FFFFFFFLL)
                return fail(QMM_ERR_UNSUPPORTED, "qmm_gemm_batch: batch too large for one launch");
            cost += b.pairs * b.tpr;
            if (b.K > max_k) max_k = b.K;
        }
        bp.total_cost = cost;
        bp.max_k = max_k;
        constexpr int WARPS = 8;
        const size_t smem = (size_t)max_k * 6 + (size_t)WARPS * 128 * sizeof(float);
        const int units = cost / (max_k / tile_k_of(fmt)) + 1;
        int grid = kNumSMs * (QMM_BATCH_THREADS_PER_SM / (WARPS * 32));
        if (units < grid) grid = units;
        void (*kern)(BatchParams) = fmt == QMM_Q4   ? gemv_batch_kernel<QMM_Q4, WARPS, true>
                                    : fmt == QMM_Q5 ? gemv_batch_kernel<QMM_Q5, WARPS, true>
                                    : fmt == QMM_Q6 ? gemv_batch_kernel<QMM_Q6, WARPS, true>
                                                    : gemv_batch_kernel<QMM_Q8, WARPS, true>;
        cudaError_t e = cudaSuccess;
        if (smem > 48 * 1024) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemm_batch shared memory size");
        e = launch_pdl(kern, dim3(grid), dim3(WARPS * 32), smem, st, bp);
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemm_batch launch");
    }
    return QMM_OK;
}

qmm_status launch_gemv(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* x, uint16_t* y,
                       void* ws, bool allow_cluster, cudaStream_t st)
{
    if (g_knobs.gemv_no_cluster) allow_cluster = false;               // tests of the two-kernel form
    const GemvPlan p = gemv_plan(fmt, N, K, allow_cluster);
    float* partial = (float*)ws;
#define QMM_GEMV_CASE(F, W) \
    if (fmt == F && p.warps == W) return launch_gemv_t<F, W>(p, packed, N, K, x, y, partial, allow_cluster, st);
    QMM_GEMV_CASE(QMM_Q4, 8)
    QMM_GEMV_CASE(QMM_Q4, 16)
    QMM_GEMV_CASE(QMM_Q8, 8)
    QMM_GEMV_CASE(QMM_Q8, 16)
    QMM_GEMV_CASE(QMM_Q5, 8)
    QMM_GEMV_CASE(QMM_Q5, 16)
    QMM_GEMV_CASE(QMM_Q6, 8)
    QMM_GEMV_CASE(QMM_Q6, 16)
#undef QMM_GEMV_CASE
    return fail(QMM_ERR_UNSUPPORTED, "qmm_gemv: no kernel for this plan");
}

}  // namespace qmm

// --------------------------------------------------------------------------
// qmm_gemv_static: the same product for callers that must not allocate.
// --------------------------------------------------------------------------

namespace qmm {

// Scratch for the split-K partial sums of qmm_gemv_static.  It lives in the
// library image: every GPU that loads libqmm holds these bytes until the
// process exits.  In host code this name is only a handle for the runtime, not
// a device address; the address each device uses is looked up once with
// cudaGetSymbolAddress (below) and that pointer is what the kernels receive.
static __device__ __align__(256) float g_gemv_static_scratch[QMM_GEMV_STATIC_SCRATCH_BYTES / sizeof(float)];

constexpr int kMaxDevices = 64;
static float* g_static_scratch_ptr[kMaxDevices];   // device address of the array, per device; nullptr = not looked up yet

// Looks up (once per device, with that device current) where the scratch array lives.
static qmm_status static_scratch_for_current_device(float** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return check_cuda(e, "qmm_gemv_static: cudaGetDevice");
    if (dev < 0 || dev >= kMaxDevices) return fail(QMM_ERR_UNSUPPORTED, "qmm_gemv_static: device index %d not supported", dev);
    float* p = __atomic_load_n(&g_static_scratch_ptr[dev], __ATOMIC_ACQUIRE);
    if (p == nullptr) {
        int major = 0, minor = 0;
        e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
        if (e == cudaSuccess) e = cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev);
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemv_static: device attributes");
        if (major != 10 || minor != 0)
            return fail(QMM_ERR_UNSUPPORTED, "qmm_gemv_static: device %d is not compute capability 10.0 (B200)", dev);
        void* addr = nullptr;
        e = cudaGetSymbolAddress(&addr, g_gemv_static_scratch);
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemv_static: cudaGetSymbolAddress");
        p = static_cast<float*>(addr);
        __atomic_store_n(&g_static_scratch_ptr[dev], p, __ATOMIC_RELEASE);   // same value from any thread
    }
    *out = p;
    return QMM_OK;
}

}  // namespace qmm

extern "C" qmm_status qmm_gemv_static(qmm_format fmt, const void* packed, int64_t N, int64_t K,
                                      const uint16_t* x_fp16, uint16_t* y_fp16, void* stream)
{
    using namespace qmm;
    if (fmt != QMM_Q4 && fmt != QMM_Q5 && fmt != QMM_Q6 && fmt != QMM_Q8)
        return fail(QMM_ERR_INVALID_ARG, "qmm_gemv_static: unknown format %d", (int)fmt);
    if (N <= 0 || K <= 0) return fail(QMM_ERR_INVALID_ARG, "qmm_gemv_static: N=%lld and K=%lld must be positive", (long long)N, (long long)K);
    if (K % 32) return fail(QMM_ERR_SHAPE, "qmm_gemv_static: K=%lld is not a multiple of the block size 32", (long long)K);
    if (K % 256 || N % 128 || K > 32768 || N > (1 << 24))
        return fail(QMM_ERR_UNSUPPORTED, "qmm_gemv_static: needs K %% 256 == 0, N %% 128 == 0, K <= 32768, N <= 2^24 (got N=%lld K=%lld)",
                    (long long)N, (long long)K);
    if (!packed || !x_fp16 || !y_fp16) return fail(QMM_ERR_INVALID_ARG, "qmm_gemv_static: null pointer");
    if ((reinterpret_cast<uintptr_t>(packed) & 31) || (reinterpret_cast<uintptr_t>(x_fp16) & 15) ||
        (reinterpret_cast<uintptr_t>(y_fp16) & 15))
        return fail(QMM_ERR_ALIGNMENT, "qmm_gemv_static: packed must be 32-byte aligned, x and y 16-byte aligned");
    const size_t need = gemv_workspace_bytes(fmt, N, K, false);       // always the two-kernel form here
    if (need > (size_t)QMM_GEMV_STATIC_SCRATCH_BYTES)
        return fail(QMM_ERR_WORKSPACE,
                    "qmm_gemv_static: this shape needs %zu bytes of split-K scratch, the built-in scratch holds %d; "
                    "use qmm_gemv with a caller-provided workspace",
                    need, (int)QMM_GEMV_STATIC_SCRATCH_BYTES);
    float* scratch = nullptr;
    const qmm_status s = static_scratch_for_current_device(&scratch);
    if (s != QMM_OK) return s;
    // Partial sums are written in full before the second stage reads them, so the
    // scratch needs no clearing between calls.
    return launch_gemv(fmt, packed, N, K, x_fp16, y_fp16, scratch, false, (cudaStream_t)stream);
}

