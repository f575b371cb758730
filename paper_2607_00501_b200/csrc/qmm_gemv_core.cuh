// qmm_gemv_core.cuh -- the inner product of the decode kernels: one 64-k (Q4) or 32-k (Q8) tile of
// two row groups times the activation vector on the warp-level tensor path, one matrix row per lane.
// Shared by the GEMV kernels (codes streamed into registers) and the chained decode kernel (codes
// staged in shared memory by bulk copies).
#pragma once

#include "qmm_common.cuh"

namespace qmm {

// D(16x8, fp32) += A(16x16, fp16, row) * B(16x8, fp16, col) on the warp-level tensor path.
__device__ __forceinline__ void mma16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Same, starting a new accumulation (C = 0) without spending instructions on zeroing registers.
__device__ __forceinline__ void mma16816_zero(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                              uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
                 : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}

// How a warp multiplies with one row per lane and no shuffles.
//
// Lane l = 4g + t holds codes of matrix row l of two row groups (P and Q) for
// the same k range.  Its pairs go into the A fragment of m16n8k16 as
//   a0/a2 -> MMA row g,   k slots {2t,2t+1} / {2t+8,2t+9}   (row group P)
//   a1/a3 -> MMA row g+8, same slots                         (row group Q)
// so MMA row g carries, in the four slot groups t = 0..3, the same four k of
// the four matrix rows 4g..4g+3.  B column j is the activation quadruple in
// slot group j and zero elsewhere, hence D[g][j] = (row 4g+j of P) . x and
// D[g+8][j] = (row 4g+j of Q) . x for j < 4.  Lanes with t < 2 receive them:
// c0,c1 = rows 4g+2t, 4g+2t+1 of P;  c2,c3 = the same rows of Q.
// Products (small integer x fp16) are exact; accumulation is fp32.

// Activations for B come from shared memory: lanes 0,5,10,15 (g == t) read x,
// every other lane reads an all-zero region of the same size, so that one
// per-lane base pointer and immediate offsets serve all loads.

// Q4: tile = 64 k.  acc[0..1] rows of P, acc[2..3] rows of Q (see above).
__device__ __forceinline__ void tile_pair_mma_q4(const u32x8& cp, const u32x8& cq, uint2 sp, uint2 sq,
                                                 const uint4* xt, float (&acc)[4], const Q4Consts& kc)
{
#pragma unroll
    for (int b = 0; b < 2; ++b) {
        float c[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 xv = xt[b * 4 + i];                      // activations k = 8(4b+i) .. +7
            __half2 p[4], q[4];
            q4_word_to_h2(cp.v[b * 4 + i], p, kc);
            q4_word_to_h2(cq.v[b * 4 + i], q, kc);
            if (i == 0)
                mma16816_zero(c, as_u32(p[0]), as_u32(q[0]), as_u32(p[1]), as_u32(q[1]), xv.x, xv.y);
            else
                mma16816(c, as_u32(p[0]), as_u32(q[0]), as_u32(p[1]), as_u32(q[1]), xv.x, xv.y);
            mma16816(c, as_u32(p[2]), as_u32(q[2]), as_u32(p[3]), as_u32(q[3]), xv.z, xv.w);
        }
        // scales: sp.x / sp.y = rows 4g+2t / 4g+2t+1 of P as (block 0, block 1) fp16 pairs
        const float dp0 = __half2float(b ? __high2half(as_h2(sp.x)) : __low2half(as_h2(sp.x)));
        const float dp1 = __half2float(b ? __high2half(as_h2(sp.y)) : __low2half(as_h2(sp.y)));
        const float dq0 = __half2float(b ? __high2half(as_h2(sq.x)) : __low2half(as_h2(sq.x)));
        const float dq1 = __half2float(b ? __high2half(as_h2(sq.y)) : __low2half(as_h2(sq.y)));
        acc[0] = fmaf(dp0, c[0], acc[0]);
        acc[1] = fmaf(dp1, c[1], acc[1]);
        acc[2] = fmaf(dq0, c[2], acc[2]);
        acc[3] = fmaf(dq1, c[3], acc[3]);
    }
}

// Q8: tile = 32 k (one block); scales are one fp16 per row: s.x low/high = rows 4g+2t, 4g+2t+1.
__device__ __forceinline__ void tile_pair_mma_q8(const u32x8& cp, const u32x8& cq, uint32_t sp, uint32_t sq,
                                                 const uint4* xt, float (&acc)[4])
{
    float c[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint4 xv = xt[i];                                  // activations k = 8i .. 8i+7
        __half2 p[2], q[2];
        q8_word_to_h2(cp.v[2 * i], p);
        q8_word_to_h2(cq.v[2 * i], q);
        if (i == 0)
            mma16816_zero(c, as_u32(p[0]), as_u32(q[0]), as_u32(p[1]), as_u32(q[1]), xv.x, xv.y);
        else
            mma16816(c, as_u32(p[0]), as_u32(q[0]), as_u32(p[1]), as_u32(q[1]), xv.x, xv.y);
        q8_word_to_h2(cp.v[2 * i + 1], p);
        q8_word_to_h2(cq.v[2 * i + 1], q);
        mma16816(c, as_u32(p[0]), as_u32(q[0]), as_u32(p[1]), as_u32(q[1]), xv.z, xv.w);
    }
    acc[0] = fmaf(__half2float(__low2half(as_h2(sp))), c[0], acc[0]);
    acc[1] = fmaf(__half2float(__high2half(as_h2(sp))), c[1], acc[1]);
    acc[2] = fmaf(__half2float(__low2half(as_h2(sq))), c[2], acc[2]);
    acc[3] = fmaf(__half2float(__high2half(as_h2(sq))), c[3], acc[3]);
}

// Q5 / Q6: a Q4 tile pair with the high-bit words of the two rows (hp, hq) merged in while unpacking.
template <int FMT, typename HI>
__device__ __forceinline__ void tile_pair_mma_q56(const u32x8& cp, const u32x8& cq, const HI& hp, const HI& hq, uint2 sp, uint2 sq,
                                                  const uint4* xt, float (&acc)[4], const Q4Consts& kc)
{
    const uint32_t* hpw = reinterpret_cast<const uint32_t*>(&hp);
    const uint32_t* hqw = reinterpret_cast<const uint32_t*>(&hq);
#pragma unroll
    for (int b = 0; b < 2; ++b) {
        float c[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int j = b * 4 + i;                             // packed word of the tile
            const int hw = FMT == QMM_Q5 ? j / 4 : j / 2;        // the high-bit word that covers it
            const uint4 xv = xt[j];                              // activations k = 8j .. 8j+7
            __half2 p[4], q[4];
            q56_word_to_h2<FMT>(cp.v[j], hpw[hw], j, p, kc);
            q56_word_to_h2<FMT>(cq.v[j], hqw[hw], j, q, kc);
            if (i == 0)
                mma16816_zero(c, as_u32(p[0]), as_u32(q[0]), as_u32(p[1]), as_u32(q[1]), xv.x, xv.y);
            else
                mma16816(c, as_u32(p[0]), as_u32(q[0]), as_u32(p[1]), as_u32(q[1]), xv.x, xv.y);
            mma16816(c, as_u32(p[2]), as_u32(q[2]), as_u32(p[3]), as_u32(q[3]), xv.z, xv.w);
        }
        const float dp0 = __half2float(b ? __high2half(as_h2(sp.x)) : __low2half(as_h2(sp.x)));
        const float dp1 = __half2float(b ? __high2half(as_h2(sp.y)) : __low2half(as_h2(sp.y)));
        const float dq0 = __half2float(b ? __high2half(as_h2(sq.x)) : __low2half(as_h2(sq.x)));
        const float dq1 = __half2float(b ? __high2half(as_h2(sq.y)) : __low2half(as_h2(sq.y)));
        acc[0] = fmaf(dp0, c[0], acc[0]);
        acc[1] = fmaf(dp1, c[1], acc[1]);
        acc[2] = fmaf(dq0, c[2], acc[2]);
        acc[3] = fmaf(dq1, c[3], acc[3]);
    }
}

template <int FMT> struct ScaleRegs { using type = uint2; };
template <> struct ScaleRegs<QMM_Q8> { using type = uint32_t; };

// High-bit words of one row of a tile (Q5: 8 bytes, Q6: 16 bytes; nothing for Q4 / Q8).
struct NoHi {};
template <int FMT> struct HiRegs { using type = NoHi; };
template <> struct HiRegs<QMM_Q5> { using type = uint2; };
template <> struct HiRegs<QMM_Q6> { using type = uint4; };

template <int FMT>
__device__ __forceinline__ typename HiRegs<FMT>::type load_hi(const uint8_t* tile, int lane)
{
    if constexpr (FMT == QMM_Q5) {
        uint2 r;
        asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(tile + kTileCodeBytes + 8 * lane));
        return r;
    } else if constexpr (FMT == QMM_Q6) {
        uint4 r;
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w)
                     : "l"(tile + kTileCodeBytes + 16 * lane));
        return r;
    } else {
        return NoHi{};
    }
}

// One tile pair of any format.
template <int FMT>
__device__ __forceinline__ void tile_pair_mma(const u32x8& cp, const u32x8& cq, const typename HiRegs<FMT>::type& hp,
                                              const typename HiRegs<FMT>::type& hq, typename ScaleRegs<FMT>::type sp,
                                              typename ScaleRegs<FMT>::type sq, const uint4* xt, float (&acc)[4], const Q4Consts& kc)
{
    if constexpr (FMT == QMM_Q4) tile_pair_mma_q4(cp, cq, sp, sq, xt, acc, kc);
    else if constexpr (FMT == QMM_Q8) tile_pair_mma_q8(cp, cq, sp, sq, xt, acc);
    else tile_pair_mma_q56<FMT>(cp, cq, hp, hq, sp, sq, xt, acc, kc);
}

// Scales of rows 4g+2(t&1) and the next row of one tile (the rows whose sums this lane receives).
template <int FMT>
__device__ __forceinline__ typename ScaleRegs<FMT>::type load_scales(const uint8_t* tile, int lane)
{
    const int row = (lane & ~3) + 2 * (lane & 1);
    if constexpr (FMT == QMM_Q8) {
        return ld_nc_u32(tile + kTileCodeBytes + 2 * row);
    } else {
        uint2 r;
        asm volatile("ld.global.nc.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(tile + Fmt<FMT>::scale_off + 4 * row));
        return r;
    }
}

// ------------------------------------------------------------ thread-block cluster helpers

// Store to the same shared-memory location in the cluster's first block.
__device__ __forceinline__ void st_cluster_rank0(float* local_ptr, float v)
{
    uint32_t local = static_cast<uint32_t>(__cvta_generic_to_shared(local_ptr)), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(remote) : "r"(local));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(v) : "memory");
}

// Barrier over all threads of the cluster (hardware barrier; the blocks of a cluster are co-scheduled).
__device__ __forceinline__ void cluster_sync()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

}  // namespace qmm
