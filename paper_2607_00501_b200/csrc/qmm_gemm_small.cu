// qmm_gemm_small.cu -- Y[M, N] = X[M, K] W^T for a handful of tokens (M <= 8): a decode step of a
// small batch, or the tail of a prefill chunk.
//
// At these sizes the product is bound by streaming W once, exactly like the single-token product
// (Sec. 3.3: decode is memory-bound), so it runs on the decode kernels' inner product rather than on
// the prefill kernel, whose 128-row tiles and fp16 expansion cost the same whatever M is: the codes are
// streamed once, unpacked once, and multiplied by all eight tokens in one warp-level MMA per 256
// weights (see FragRegs).
//
// Work item = (pair of row groups, K split): 64 outputs for every token; the block's warps split the
// item's K range, their sums are added in warp order.  K is split across blocks only when the row
// groups alone cannot cover the SMs; the blocks of an item are then a thread-block cluster and add
// their sums through the shared memory of its first block, in split order: no workspace, no second
// launch, the same bits on every call.
#include "qmm_gemv_core.cuh"

namespace qmm {

constexpr int kSmallWarps = 8;
constexpr int kSmallMaxSplits = 8;          // portable cluster size
constexpr int kSmallMaxTokens = 8;          // one group of eight tokens per MMA

// How a warp multiplies a tile pair by up to eight tokens with one MMA per 256 weights.
//
// The single-token kernels give every lane one matrix row and pay for it with a sparse B operand.
// Here every lane still moves its own row of the tile (32 contiguous bytes), but into shared memory,
// transposed on the way: ldmatrix then hands lane l = 4g + t, of each of the four rows 4g .. 4g+3 of
// both row groups (P, Q), the packed words t and t + 4: one 8-k chunk of each 32-element block (Q8:
// 4-k chunks of the tile's one block).  For row i of the four, the lane's words are then exactly its share of a 16 x 16
// A fragment whose MMA row g is matrix row 4g+i of P, MMA row g+8 the same row of Q, and whose 16 k
// are the chunk t of every lane t -- all inside one quantisation block, so the block's scale still
// multiplies the fp32 sum afterwards and the integer products stay exact.  B is dense: lane (g, t)
// supplies token g's activations for chunk t (one 16-byte load per block, shared by the four rows).  D[g][2t, 2t+1] / D[g+8][..] are row 4g+i of P / Q for tokens 2t, 2t+1.
template <int FMT>
struct SmallSlot {                                              // what a lane needs of a tile pair beside the codes
    static constexpr int HW = FMT == QMM_Q5 || FMT == QMM_Q6 ? 2 : 0;
    uint32_t hp[4][HW ? HW : 1], hq[4][HW ? HW : 1];            // high-bit words covering words t, t+4 of rows 4g+i (Q5 / Q6)
    uint32_t sp[FMT == QMM_Q8 ? 2 : 4], sq[FMT == QMM_Q8 ? 2 : 4];   // scales of rows 4g .. 4g+3 (fp16; Q8: one per row, else two)
};

template <int FMT>
struct FragRegs {
    uint32_t wp[4][2], wq[4][2];                                // [row i][block b]: word t + 4b of row 4g+i
};

__device__ __forceinline__ uint2 ld_nc_u32x2(const void* p)
{
    uint2 r;
    asm volatile("ld.global.nc.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p));
    return r;
}
__device__ __forceinline__ uint4 ld_nc_u32x4(const void* p)
{
    uint4 r;
    asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// The transposition.  Row r of a tile is stored as two 16-byte halves at
// 128 (r / 4) + 16 ((2 (r % 4) + h) ^ (r / 4)): the XOR spreads the eight rows that one ldmatrix matrix
// reads (rows 4g+i, g = 0..7, same i and h) over all banks.  Matrix (i, h) of eight 16-byte rows then
// gives lane (g, t) the 32-bit word t of half h of row 4g+i.
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& d0, uint32_t& d1, uint32_t& d2, uint32_t& d3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(d0), "=r"(d1), "=r"(d2), "=r"(d3) : "r"(addr) : "memory");
}

// q56_word_to_h2 for a word whose index within its high-bit word (jq = j & 3 for Q5, j & 1 for Q6) is
// known only at run time: the high-bit word is first shifted down to that word's bits, the per-pair
// shifts are then constants.
template <int FMT>
__device__ __forceinline__ void q56_word_to_h2_dyn(uint32_t w, uint32_t H, int jq, __half2 (&q)[4], const Q4Consts& k)
{
    constexpr bool Q5 = FMT == QMM_Q5;
    const __half2 c_lo = as_h2(Q5 ? 0x64106410u : 0x64206420u);          // 1040 / 1056
    const __half2 c16th = as_h2(0x2C002C00u);
    const __half2 c_hi = as_h2(Q5 ? 0xD500D500u : 0xD600D600u);          // -80 / -96
    const uint32_t m_lo = Q5 ? 0x00100010u : 0x00300030u, m_hi = Q5 ? 0x01000100u : 0x03000300u;
    const uint32_t w8 = w >> 8;
    const uint32_t Hs = H >> (Q5 ? 4 * jq : 8 * jq);
    auto hi_at = [&](int p, int target) -> uint32_t {                      // pair p's high bits moved to bit `target`
        const int s = (Q5 ? p : 2 * p) - target;
        return s >= 0 ? Hs >> s : Hs << -s;
    };
    q[0] = __hsub2(as_h2(and_or(hi_at(0, 4), m_lo, and_or(w, k.mask_lo, k.magic))), c_lo);
    q[1] = __hfma2(as_h2(and_or(hi_at(1, 8), m_hi, and_or(w, k.mask_hi, k.magic))), c16th, c_hi);
    q[2] = __hsub2(as_h2(and_or(hi_at(2, 4), m_lo, and_or(w8, k.mask_lo, k.magic))), c_lo);
    q[3] = __hfma2(as_h2(and_or(hi_at(3, 8), m_hi, and_or(w8, k.mask_hi, k.magic))), c16th, c_hi);
}

// One tile pair times the lane's activations (xr[b][n]: block b, token group n).
// acc[n][i][0..1]: row 4g+i of P for tokens 8n+2t, 8n+2t+1; acc[n][i][2..3]: the same row of Q.
template <int FMT, int NG>
__device__ __forceinline__ void frag_mma_x(const SmallSlot<FMT>& r, const FragRegs<FMT>& f, const uint4 (&xr)[FMT == QMM_Q8 ? 1 : 2][NG], int t,
                                         float (&acc)[NG][4][4], const Q4Consts& kc)
{
    constexpr int BLOCKS = FMT == QMM_Q8 ? 1 : 2;
#pragma unroll
    for (int b = 0; b < BLOCKS; ++b) {
        uint4 xv[NG];
#pragma unroll
        for (int n = 0; n < NG; ++n) xv[n] = xr[b][n];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __half2 p[4], q[4];
            if constexpr (FMT == QMM_Q8) {
                __half2 a[2];
                q8_word_to_h2(f.wp[i][0], a);
                p[0] = a[0], p[1] = a[1];
                q8_word_to_h2(f.wp[i][1], a);
                p[2] = a[0], p[3] = a[1];
                q8_word_to_h2(f.wq[i][0], a);
                q[0] = a[0], q[1] = a[1];
                q8_word_to_h2(f.wq[i][1], a);
                q[2] = a[0], q[3] = a[1];
            } else if constexpr (FMT == QMM_Q4) {
                q4_word_to_h2(f.wp[i][b], p, kc);
                q4_word_to_h2(f.wq[i][b], q, kc);
            } else {
                // word j = t + 4b of the row; only j's position inside its high-bit word matters
                const int jq = FMT == QMM_Q5 ? (t & 3) : (t & 1);
                q56_word_to_h2_dyn<FMT>(f.wp[i][b], r.hp[i][b], jq, p, kc);
                q56_word_to_h2_dyn<FMT>(f.wq[i][b], r.hq[i][b], jq, q, kc);
            }
            float dp, dq;
            if constexpr (FMT == QMM_Q8) {
                const __half2 hp2 = as_h2(r.sp[i >> 1]), hq2 = as_h2(r.sq[i >> 1]);
                dp = __half2float((i & 1) ? __high2half(hp2) : __low2half(hp2));
                dq = __half2float((i & 1) ? __high2half(hq2) : __low2half(hq2));
            } else {
                dp = __half2float(b ? __high2half(as_h2(r.sp[i])) : __low2half(as_h2(r.sp[i])));
                dq = __half2float(b ? __high2half(as_h2(r.sq[i])) : __low2half(as_h2(r.sq[i])));
            }
#pragma unroll
            for (int n = 0; n < NG; ++n) {
                float c[4];
                mma16816_zero(c, as_u32(p[0]), as_u32(q[0]), as_u32(p[1]), as_u32(q[1]), xv[n].x, xv[n].y);
                mma16816(c, as_u32(p[2]), as_u32(q[2]), as_u32(p[3]), as_u32(q[3]), xv[n].z, xv[n].w);
                acc[n][i][0] = fmaf(dp, c[0], acc[n][i][0]);
                acc[n][i][1] = fmaf(dp, c[1], acc[n][i][1]);
                acc[n][i][2] = fmaf(dq, c[2], acc[n][i][2]);
                acc[n][i][3] = fmaf(dq, c[3], acc[n][i][3]);
            }
        }
    }
}

// ------------------------------------------------------------------ the ring
//
// The tile pairs in flight are held in shared memory, not in registers: every warp owns a ring of
// few slots and fills them with 16-byte asynchronous copies -- each lane copies the two halves
// of its row straight to their transposed places, the first lanes the scale (and high-bit) planes as
// they are -- one commit group per tile pair.  Nothing is held in registers while the copies fly, so
// the ring is deep and the loop needs no register double buffer; the copies of the block's next work
// item run under the reduction of the current one.

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 r;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr)
{
    uint2 r;
    asm volatile("ld.shared.v2.b32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "r"(addr));
    return r;
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t r;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(r) : "r"(addr));
    return r;
}

// One tile pair -> one slot (2 * tile bytes: P then Q; the first 1024 bytes of each transposed).
template <int FMT>
__device__ __forceinline__ void ring_issue(uint32_t slot, const uint8_t* tile_p, const uint8_t* tile_q, int lane)
{
    constexpr int TB = Fmt<FMT>::tile_bytes;
    constexpr int EX = (TB - kTileCodeBytes) / 16;              // 16-byte chunks behind the codes
    const int wg = lane >> 2, wi = lane & 3;
    const uint32_t st0 = slot + 128 * wg + 16 * ((2 * wi) ^ wg), st1 = slot + 128 * wg + 16 * ((2 * wi + 1) ^ wg);
    cp_async16(st0, tile_p + 32 * lane);
    cp_async16(st1, tile_p + 32 * lane + 16);
    cp_async16(st0 + TB, tile_q + 32 * lane);
    cp_async16(st1 + TB, tile_q + 32 * lane + 16);
#pragma unroll
    for (int c0 = 0; c0 < EX; c0 += 32) {
        const int c = c0 + lane;
        if (c < EX) {
            cp_async16(slot + kTileCodeBytes + 16 * c, tile_p + kTileCodeBytes + 16 * c);
            cp_async16(slot + TB + kTileCodeBytes + 16 * c, tile_q + kTileCodeBytes + 16 * c);
        }
    }
}

// Slot -> registers: the lane's share of the A fragments, the scales and high-bit words of its rows.
template <int FMT>
__device__ __forceinline__ void ring_read(uint32_t slot, SmallSlot<FMT>& r, FragRegs<FMT>& f, int lane)
{
    constexpr int TB = Fmt<FMT>::tile_bytes;
    const int g = lane >> 2, t = lane & 3;
    const int mg = lane & 7, mj = lane >> 3;                    // ldmatrix: this lane addresses row mg of matrix mj
    const uint32_t ld0 = slot + 128 * mg + 16 * ((2 * mj) ^ mg), ld1 = slot + 128 * mg + 16 * ((2 * mj + 1) ^ mg);
    ldmatrix_x4(ld0, f.wp[0][0], f.wp[1][0], f.wp[2][0], f.wp[3][0]);
    ldmatrix_x4(ld1, f.wp[0][1], f.wp[1][1], f.wp[2][1], f.wp[3][1]);
    ldmatrix_x4(ld0 + TB, f.wq[0][0], f.wq[1][0], f.wq[2][0], f.wq[3][0]);
    ldmatrix_x4(ld1 + TB, f.wq[0][1], f.wq[1][1], f.wq[2][1], f.wq[3][1]);
    if constexpr (FMT == QMM_Q8) {
        const uint2 a = lds64(slot + Fmt<FMT>::scale_off + 8 * g), b = lds64(slot + TB + Fmt<FMT>::scale_off + 8 * g);
        r.sp[0] = a.x, r.sp[1] = a.y, r.sq[0] = b.x, r.sq[1] = b.y;
    } else {
        const uint4 a = lds128(slot + Fmt<FMT>::scale_off + 16 * g), b = lds128(slot + TB + Fmt<FMT>::scale_off + 16 * g);
        r.sp[0] = a.x, r.sp[1] = a.y, r.sp[2] = a.z, r.sp[3] = a.w;
        r.sq[0] = b.x, r.sq[1] = b.y, r.sq[2] = b.z, r.sq[3] = b.w;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = 4 * g + i;
        if constexpr (FMT == QMM_Q5) {
            const uint2 a = lds64(slot + kTileCodeBytes + 8 * row), b = lds64(slot + TB + kTileCodeBytes + 8 * row);
            r.hp[i][0] = a.x, r.hp[i][1] = a.y, r.hq[i][0] = b.x, r.hq[i][1] = b.y;
        } else if constexpr (FMT == QMM_Q6) {
            r.hp[i][0] = lds32(slot + kTileCodeBytes + 16 * row + 4 * (t >> 1));
            r.hp[i][1] = lds32(slot + kTileCodeBytes + 16 * row + 4 * (t >> 1) + 8);
            r.hq[i][0] = lds32(slot + TB + kTileCodeBytes + 16 * row + 4 * (t >> 1));
            r.hq[i][1] = lds32(slot + TB + kTileCodeBytes + 16 * row + 4 * (t >> 1) + 8);
        }
    }
}

// Ring depth and resident blocks per SM.  One product at a time (gemm_small_kernel): 4 slots, 2 blocks of
// 128 registers for every format.  The batched launch: the same for the 4-bit formats, which are bound by
// instruction issue; Q8, bound by memory latency, runs 3 blocks with 2 slots each (measured both ways;
// for single products chained on a stream that geometry was slower).
constexpr int kDenseStages = 4;
template <int FMT> struct SmallGeom { static constexpr int kStages = 4, kBlocks = 2; };
template <> struct SmallGeom<QMM_Q8> { static constexpr int kStages = 2, kBlocks = 3; };

// Dynamic shared memory: WARPS * kStages slots, WARPS * 8*NG * 64 floats for the warps' sums, and
// (cluster form, used in the first block) 2 * splits * 8*NG * 64 floats.
template <int FMT, int NG>
__global__ void __launch_bounds__(kSmallWarps * 32, 2)
gemm_small_kernel(const uint8_t* __restrict__ packed, const uint16_t* __restrict__ X, int64_t ldx,
                       uint16_t* __restrict__ Y, int64_t ldy, int M, int K, int tiles_per_row, int splits, int items)
{
    constexpr int WARPS = kSmallWarps, NT = 8 * NG, kStages = kDenseStages;
    constexpr int TB = Fmt<FMT>::tile_bytes;
    constexpr int SLOT = 2 * TB;
    extern __shared__ uint4 smem[];
    const int tps = tiles_per_row / splits;                     // tiles per item
    float* red = reinterpret_cast<float*>(smem + WARPS * kStages * SLOT / 16);   // behind the rings
    float* cred = red + WARPS * NT * 64;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const bool clustered = splits > 1;
    int cluster_round = 0;
    const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(smem)) + warp * (kStages * SLOT);

    const size_t group_bytes = (size_t)tiles_per_row * TB;
    const int s = blockIdx.x % splits;                          // the same for every item of this block (grid = whole clusters)
    const int t_begin = s * tps + warp, t_end = (s + 1) * tps;
    const bool has_tiles = warp < tps;

    // producer: runs kStages tile pairs ahead of the consumer, across work items
    int p_item = blockIdx.x, p_t = t_begin;
    auto produce = [&](int stage) {
        if (has_tiles && p_item < items) {
            const uint8_t* tp = packed + (size_t)(2 * (p_item / splits)) * group_bytes + (size_t)p_t * TB;
            ring_issue<FMT>(ring + stage * SLOT, tp, tp + group_bytes, lane);
            p_t += WARPS;
            if (p_t >= t_end) {
                p_item += gridDim.x;
                p_t = t_begin;
            }
        }
        cp_async_commit();                                      // one group per call, empty or not
    };
#pragma unroll
    for (int st = 0; st < kStages; ++st) produce(st);       // weights never depend on the previous kernel

    pdl_launch_dependents();
    pdl_wait();                                                 // X may come from the previous kernel
    // activations come straight from global memory (they are few and shared by every warp: L1 / L2 hits):
    // lane (g, t) reads token g's chunk t of each 32-element block, lanes of tokens that do not exist read nothing
    const uint16_t* xrow[NG];
#pragma unroll
    for (int n = 0; n < NG; ++n) xrow[n] = 8 * n + g < M ? X + (size_t)(8 * n + g) * ldx : nullptr;
    auto load_x = [&](int tt, uint4 (&xr)[FMT == QMM_Q8 ? 1 : 2][NG]) {
#pragma unroll
        for (int b = 0; b < (FMT == QMM_Q8 ? 1 : 2); ++b)
#pragma unroll
            for (int n = 0; n < NG; ++n) {
                xr[b][n] = make_uint4(0u, 0u, 0u, 0u);
                if (xrow[n]) {
                    const uint16_t* xt = xrow[n] + (size_t)tt * Fmt<FMT>::tile_k;
                    if constexpr (FMT == QMM_Q8) {
                        // words t and 4 + t of the row are k = 4t .. 4t+3 and 16 + 4t .. 16 + 4t+3 of the tile
                        const uint2 lo = ld_nc_u32x2(xt + 4 * t4), hi = ld_nc_u32x2(xt + 16 + 4 * t4);
                        xr[b][n] = make_uint4(lo.x, lo.y, hi.x, hi.y);
                    } else {
                        xr[b][n] = ld_nc_u32x4(xt + 32 * b + 8 * t4);
                    }
                }
            }
    };
    Q4Consts kc;
    kc.init();

    int stage = 0;
    for (int item = blockIdx.x; item < items; item += gridDim.x) {
        const int pair = item / splits;
        float acc[NG][4][4];
#pragma unroll
        for (int n = 0; n < NG; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[n][i][0] = acc[n][i][1] = acc[n][i][2] = acc[n][i][3] = 0.f;
        if (has_tiles) {
            for (int tt = t_begin; tt < t_end; tt += WARPS) {
                uint4 xr[FMT == QMM_Q8 ? 1 : 2][NG];
                load_x(tt, xr);                                 // in flight while the tile pair lands
                cp_async_wait<kStages - 1>();               // the oldest group -- this tile pair -- has landed
                __syncwarp();
                SmallSlot<FMT> r;
                FragRegs<FMT> f;
                ring_read<FMT>(ring + stage * SLOT, r, f, lane);
                __syncwarp();                                   // every lane has read the slot
                produce(stage);
                frag_mma_x<FMT, NG>(r, f, xr, t4, acc, kc);
                stage = stage + 1 == kStages ? 0 : stage + 1;
            }
        }
        // red[warp][token][64]: rows 0..31 of P, then of Q
#pragma unroll
        for (int n = 0; n < NG; ++n)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                float* w = red + (warp * NT + 8 * n + 2 * t4) * 64 + 4 * g + i;
                w[0] = acc[n][i][0];
                w[64] = acc[n][i][1];
                w[32] = acc[n][i][2];
                w[64 + 32] = acc[n][i][3];
            }
        __syncthreads();
        const int live = (M < NT ? M : NT) * 64;                // sums of tokens that exist
        if (!clustered) {
            for (int i = threadIdx.x; i < live; i += WARPS * 32) {
                float sum = red[i];
#pragma unroll
                for (int w = 1; w < WARPS; ++w) sum += red[w * NT * 64 + i];
                Y[(size_t)(i >> 6) * ldy + pair * 64 + (i & 63)] = __half_as_ushort(__float2half_rn(sum));
            }
        } else {
            float* slot = cred + (cluster_round & 1) * (splits * NT * 64);
            for (int i = threadIdx.x; i < live; i += WARPS * 32) {
                float sum = red[i];
#pragma unroll
                for (int w = 1; w < WARPS; ++w) sum += red[w * NT * 64 + i];
                st_cluster_rank0(slot + s * NT * 64 + i, sum);
            }
            cluster_sync();
            if (s == 0) {
                for (int i = threadIdx.x; i < live; i += WARPS * 32) {
                    float total = slot[i];
                    for (int sp = 1; sp < splits; ++sp) total += slot[sp * NT * 64 + i];
                    Y[(size_t)(i >> 6) * ldy + pair * 64 + (i & 63)] = __half_as_ushort(__float2half_rn(total));
                }
            }
            ++cluster_round;
        }
        __syncthreads();
    }
    cp_async_wait<0>();                                         // (only empty groups can be left)
}

// ------------------------------------------------------------------ batch
//
// Many independent few-token products in ONE launch -- every matrix of a decode step for a batch of
// up to eight sequences (the paper's decode gains come from fewer, fused dispatches, Sec. 3.3).
// As in gemv_batch_kernel: work unit = (problem, pair of row groups), the unit list is cut into
// gridDim.x contiguous ranges of equal cost (tiles), so blocks finish together although problems
// differ in K; no K split across blocks, no workspace.  The ring runs on across units and problems.
constexpr int kSmallMaxBatch = 128;

struct SmallBatchProblem {
    const uint8_t* packed;
    const uint16_t* X;        // [M, ldx]
    uint16_t* Y;              // [M, ldy]
    int ldx, ldy;
    int tpr;                  // tiles per row
    int pairs;                // N / 64
    int cost_begin;           // tiles of all earlier problems
};

struct SmallBatchParams {
    int count, total_cost, M;
    SmallBatchProblem p[kSmallMaxBatch];
};

template <int FMT>
__global__ void __launch_bounds__(kSmallWarps * 32, SmallGeom<FMT>::kBlocks)
gemm_small_batch_kernel(const __grid_constant__ SmallBatchParams bp)
{
    constexpr int WARPS = kSmallWarps, kSBStages = SmallGeom<FMT>::kStages;
    constexpr int TB = Fmt<FMT>::tile_bytes, TK = Fmt<FMT>::tile_k;
    constexpr int SLOT = 2 * TB;
    extern __shared__ uint4 smem[];
    float* red_all = reinterpret_cast<float*>(smem + WARPS * kSBStages * SLOT / 16);   // [2][WARPS][8][64], behind the rings
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t4 = lane & 3;
    const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(smem)) + warp * (kSBStages * SLOT);
    const int M = bp.M;

    // this block's range of the unit list, by cost; a unit belongs to the block whose range holds its first tile
    const int c0 = (int)(((long long)bp.total_cost * blockIdx.x) / gridDim.x);
    const int c1 = (int)(((long long)bp.total_cost * (blockIdx.x + 1)) / gridDim.x);
    int pi0 = 0;
    while (pi0 < bp.count && bp.p[pi0].cost_begin + bp.p[pi0].pairs * bp.p[pi0].tpr <= c0) ++pi0;
    int unit0 = 0;
    if (pi0 < bp.count) {
        const int rel = c0 - bp.p[pi0].cost_begin;
        unit0 = rel <= 0 ? 0 : (rel + bp.p[pi0].tpr - 1) / bp.p[pi0].tpr;
        if (unit0 >= bp.p[pi0].pairs) {
            ++pi0;
            unit0 = 0;
        }
    }
    auto valid = [&](int p, int u) { return p < bp.count && bp.p[p].cost_begin + u * bp.p[p].tpr < c1; };

    // producer: runs kSBStages tile pairs ahead of the consumer, across units and problems
    int p_pi = pi0, p_unit = unit0, p_left = 0;                 // p_left: this warp's tiles still to request in the unit
    const uint8_t* p_tp = nullptr;
    size_t p_gb = 0;
    auto p_open = [&]() {                                       // the first unit from (p_pi, p_unit) on in which this warp has tiles
        while (valid(p_pi, p_unit)) {
            const int tpr = bp.p[p_pi].tpr;
            if (warp < tpr) {
                p_gb = (size_t)tpr * TB;
                p_tp = bp.p[p_pi].packed + (size_t)(2 * p_unit) * p_gb + (size_t)warp * TB;
                p_left = (tpr - warp + WARPS - 1) / WARPS;
                return;
            }
            if (++p_unit >= bp.p[p_pi].pairs) {
                ++p_pi;
                p_unit = 0;
            }
        }
        p_left = 0;
    };
    p_open();
    auto produce = [&](int stage) {
        if (p_left) {
            ring_issue<FMT>(ring + stage * SLOT, p_tp, p_tp + p_gb, lane);
            p_tp += WARPS * TB;
            if (--p_left == 0) {
                if (++p_unit >= bp.p[p_pi].pairs) {
                    ++p_pi;
                    p_unit = 0;
                }
                p_open();
            }
        }
        cp_async_commit();                                      // one group per call, empty or not
    };
#pragma unroll
    for (int st = 0; st < kSBStages; ++st) produce(st);       // weights never depend on the previous kernel

    pdl_launch_dependents();
    pdl_wait();                                                 // activations may come from the previous kernel
    Q4Consts kc;
    kc.init();

    int stage = 0, round = 0;
    int pi = pi0, unit = unit0;
    while (valid(pi, unit)) {
        float* red = red_all + (round & 1) * (WARPS * 8 * 64);
        const int tpr = bp.p[pi].tpr;
        const uint16_t* xrow = g < M ? bp.p[pi].X + (size_t)g * bp.p[pi].ldx : nullptr;
        float acc[1][4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i) acc[0][i][0] = acc[0][i][1] = acc[0][i][2] = acc[0][i][3] = 0.f;
        for (int tt = warp; tt < tpr; tt += WARPS) {
            uint4 xr[FMT == QMM_Q8 ? 1 : 2][1];
#pragma unroll
            for (int b = 0; b < (FMT == QMM_Q8 ? 1 : 2); ++b) {
                xr[b][0] = make_uint4(0u, 0u, 0u, 0u);
                if (xrow) {
                    const uint16_t* xt = xrow + (size_t)tt * TK;
                    if constexpr (FMT == QMM_Q8) {
                        const uint2 lo = ld_nc_u32x2(xt + 4 * t4), hi = ld_nc_u32x2(xt + 16 + 4 * t4);
                        xr[b][0] = make_uint4(lo.x, lo.y, hi.x, hi.y);
                    } else {
                        xr[b][0] = ld_nc_u32x4(xt + 32 * b + 8 * t4);
                    }
                }
            }
            cp_async_wait<kSBStages - 1>();                   // the oldest group -- this tile pair -- has landed
            __syncwarp();
            SmallSlot<FMT> r;
            FragRegs<FMT> f;
            ring_read<FMT>(ring + stage * SLOT, r, f, lane);
            __syncwarp();                                       // every lane has read the slot
            produce(stage);
            frag_mma_x<FMT, 1>(r, f, xr, t4, acc, kc);
            stage = stage + 1 == kSBStages ? 0 : stage + 1;
        }
        // red[warp][token][64]: rows 0..31 of P, then of Q
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float* w = red + (warp * 8 + 2 * t4) * 64 + 4 * g + i;
            w[0] = acc[0][i][0];
            w[64] = acc[0][i][1];
            w[32] = acc[0][i][2];
            w[64 + 32] = acc[0][i][3];
        }
        // one barrier per unit: this buffer is rewritten two units on, after every thread has passed the
        // next unit's barrier, i.e. has finished reading it
        __syncthreads();
        const int nw = tpr < WARPS ? tpr : WARPS;               // warps that had tiles (the others hold zeros)
        for (int i = threadIdx.x; i < M * 64; i += WARPS * 32) {
            float sum = red[i];
            for (int w = 1; w < nw; ++w) sum += red[w * 8 * 64 + i];
            bp.p[pi].Y[(size_t)(i >> 6) * bp.p[pi].ldy + unit * 64 + (i & 63)] = __half_as_ushort(__float2half_rn(sum));
        }
        ++round;
        if (++unit >= bp.p[pi].pairs) {
            ++pi;
            unit = 0;
        }
    }
    cp_async_wait<0>();                                         // (only empty groups can be left)
}

// ------------------------------------------------------------------ host

bool gemm_small_supported(int fmt, int64_t M)
{
    (void)fmt;
    return M >= 1 && M <= kSmallMaxTokens && !g_knobs.gemm_no_small;
}

qmm_status launch_gemv(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* x, uint16_t* y,
                       void* ws, bool allow_cluster, cudaStream_t st);
size_t gemv_workspace_bytes(int fmt, int64_t N, int64_t K, bool allow_cluster);
bool gemv_two_supported(int fmt, int64_t N, int64_t K);
qmm_status launch_gemv_two(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* X, int64_t ldx, uint16_t* Y,
                           int64_t ldy, cudaStream_t st);

struct SmallPlan {
    int splits, grid;
    size_t smem;
};

static SmallPlan small_plan(int fmt, int64_t M, int64_t N, int64_t K)
{
    const int ng = (int)((M + 7) / 8), nt = 8 * ng;
    const int tpr = (int)(K / tile_k_of(fmt));
    const int pairs = (int)(N / 64);
    const int per_sm = 2, stages = kDenseStages;
    auto smem_of = [&](int splits) {
        return (size_t)kSmallWarps * stages * 2 * tile_bytes_of(fmt) + (size_t)kSmallWarps * nt * 64 * sizeof(float) +
               (splits > 1 ? (size_t)2 * splits * nt * 64 * sizeof(float) : 0);
    };
    int splits = 1;
    // split K while the pairs alone leave SMs without a block, every warp keeps a tile, and the cluster stays small
    while (pairs * splits < kNumSMs * per_sm && tpr % (splits * 2) == 0 && tpr / (splits * 2) >= kSmallWarps / 2 && splits < 4) splits *= 2;
    SmallPlan p;
    p.splits = splits;
    p.smem = smem_of(splits);
    const int items = pairs * splits;
    const int cap = kNumSMs * per_sm / splits * splits;
    p.grid = items < cap ? items : cap;
    return p;
}

template <int FMT, int NG>
static qmm_status launch_small_t(const SmallPlan& p, const void* packed, int64_t N, int64_t K, const uint16_t* X, int64_t ldx,
                                 uint16_t* Y, int64_t ldy, int64_t M, cudaStream_t st)
{
    auto kern = gemm_small_kernel<FMT, NG>;
    if (p.smem > 227 * 1024) return fail(QMM_ERR_UNSUPPORTED, "qmm_gemm: K=%lld is too large for the few-token kernel", (long long)K);
    if (p.smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem);
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemm few-token kernel shared memory size");
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)p.grid);
    cfg.blockDim = dim3(kSmallWarps * 32);
    cfg.dynamicSmemBytes = p.smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = (unsigned)p.splits;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.splits > 1 ? 2 : 1;
    const int tpr = (int)(K / Fmt<FMT>::tile_k);
    const int items = (int)(N / 64) * p.splits;
    return check_cuda(cudaLaunchKernelEx(&cfg, kern, (const uint8_t*)packed, X, ldx, Y, ldy, (int)M, (int)K, tpr, p.splits, items),
                      "qmm_gemm few-token kernel launch");
}

qmm_status launch_gemm_small(int fmt, const void* packed, int64_t N, int64_t K, const uint16_t* X, int64_t ldx,
                             uint16_t* Y, int64_t ldy, int64_t M, cudaStream_t st)
{
    // one token: the single-token kernel (its cluster form needs no workspace)
    if (M == 1 && gemv_workspace_bytes(fmt, N, K, true) == 0) return launch_gemv(fmt, packed, N, K, X, Y, nullptr, true, st);
    // two tokens: the same kernel, the second token in the half of the MMAs' B operand it leaves idle
    if (M == 2 && gemv_two_supported(fmt, N, K)) {
        const qmm_status s2 = launch_gemv_two(fmt, packed, N, K, X, ldx, Y, ldy, st);
        if (s2 != QMM_ERR_UNSUPPORTED) return s2;
    }
    const SmallPlan p = small_plan(fmt, M, N, K);
    const int ng = (int)((M + 7) / 8);
#define QMM_SMALL_CASE(F, G) \
    if (fmt == F && ng == G) return launch_small_t<F, G>(p, packed, N, K, X, ldx, Y, ldy, M, st);
    QMM_SMALL_CASE(QMM_Q4, 1)
    QMM_SMALL_CASE(QMM_Q8, 1)
    QMM_SMALL_CASE(QMM_Q5, 1)
    QMM_SMALL_CASE(QMM_Q6, 1)
#undef QMM_SMALL_CASE
    return fail(QMM_ERR_UNSUPPORTED, "qmm_gemm: no few-token kernel for format %d, M=%lld", fmt, (long long)M);
}

// Host side of qmm_gemm_batch: up to kSmallMaxBatch problems per launch.
qmm_status launch_gemv_batch(int fmt, const qmm_gemv_problem* probs, int count, cudaStream_t st, bool out_f32);

qmm_status launch_gemv_batch_two(int fmt, const qmm_gemm_problem* probs, int count, cudaStream_t st);

qmm_status launch_gemm_small_batch(int fmt, const qmm_gemm_problem* probs, int count, int64_t M, cudaStream_t st)
{
    if (M == 2) {
        // two tokens: the single-token batched kernel carries the second token in the idle half of its
        // MMAs' B operand (activations staged in shared memory: K <= 32768)
        bool fits = true;
        for (int i = 0; i < count; ++i) fits = fits && probs[i].K <= 32768;
        if (fits) return launch_gemv_batch_two(fmt, probs, count, st);
    }
    if (M == 1) {
        // one token: the single-token batched kernel (its activations are staged in shared memory: K <= 32768)
        bool fits = true;
        for (int i = 0; i < count; ++i) fits = fits && probs[i].K <= 32768;
        if (fits) {
            for (int first = 0; first < count; first += kSmallMaxBatch) {
                const int n = count - first < kSmallMaxBatch ? count - first : kSmallMaxBatch;
                qmm_gemv_problem v[kSmallMaxBatch];
                for (int i = 0; i < n; ++i) {
                    const qmm_gemm_problem& q = probs[first + i];
                    v[i].packed = q.packed;
                    v[i].x_fp16 = q.X_fp16;
                    v[i].y_fp16 = q.Y_fp16;
                    v[i].N = q.N;
                    v[i].K = q.K;
                }
                const qmm_status s = launch_gemv_batch(fmt, v, n, st, false);
                if (s != QMM_OK) return s;
            }
            return QMM_OK;
        }
    }
    for (int first = 0; first < count; first += kSmallMaxBatch) {
        const int n = count - first < kSmallMaxBatch ? count - first : kSmallMaxBatch;
        SmallBatchParams bp = {};
        bp.count = n;
        bp.M = (int)M;
        long long cost = 0;
        int units = 0;
        for (int i = 0; i < n; ++i) {
            const qmm_gemm_problem& q = probs[first + i];
            SmallBatchProblem& b = bp.p[i];
            b.packed = (const uint8_t*)q.packed;
            b.X = q.X_fp16;
            b.Y = q.Y_fp16;
            b.ldx = (int)q.ldx;
            b.ldy = (int)q.ldy;
            b.tpr = (int)(q.K / tile_k_of(fmt));
            b.pairs = (int)(q.N / 64);
            b.cost_begin = (int)cost;
            cost += (long long)b.pairs * b.tpr;
            units += b.pairs;
            if (cost > 0x7FFFFFFFLL) return fail(QMM_ERR_UNSUPPORTED, "qmm_gemm_batch: batch too large for one launch");
        }
        bp.total_cost = (int)cost;
        const int stages = fmt == QMM_Q8 ? SmallGeom<QMM_Q8>::kStages : SmallGeom<QMM_Q4>::kStages;
        const int blocks = fmt == QMM_Q8 ? SmallGeom<QMM_Q8>::kBlocks : SmallGeom<QMM_Q4>::kBlocks;
        const size_t smem = (size_t)kSmallWarps * stages * 2 * tile_bytes_of(fmt) + (size_t)2 * kSmallWarps * 8 * 64 * sizeof(float);
        int grid = blocks * kNumSMs;
        if (units < grid) grid = units;
        void (*kern)(SmallBatchParams) = fmt == QMM_Q4   ? gemm_small_batch_kernel<QMM_Q4>
                                         : fmt == QMM_Q5 ? gemm_small_batch_kernel<QMM_Q5>
                                         : fmt == QMM_Q6 ? gemm_small_batch_kernel<QMM_Q6>
                                                         : gemm_small_batch_kernel<QMM_Q8>;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemm_batch shared memory size");
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3(kSmallWarps * 32);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        e = cudaLaunchKernelEx(&cfg, kern, bp);
        if (e != cudaSuccess) return check_cuda(e, "qmm_gemm_batch launch");
    }
    return QMM_OK;
}

}  // namespace qmm
