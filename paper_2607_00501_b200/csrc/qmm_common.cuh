// qmm_common.cuh -- device layout of packed weights and small device helpers
// shared by the kernels of libqmm (sm_100a only).
//
// Device layout ("row-group tiles").  Rows are taken in groups of 32 (one row
// per lane of a warp, and one row per lane of tensor memory in the GEMM).
// For each row group the K axis is cut into tiles; the tiles of one row group
// are consecutive in memory, row groups follow each other.
//
//   Q4 tile = 64 weights per row (two quantisation blocks), 1152 bytes:
//     [32 rows][32 B codes]  row r at byte 32 r: eight 32-bit words; word j
//                            holds elements k = 8j .. 8j+7 of the tile as
//                            nibbles u = q + 8 in the order 0,2,4,6,1,3,5,7
//                            (low nibble first), so (word >> 4p) & 0x000F000F
//                            is the pair (k = 8j+2p, 8j+2p+1) in the low/high
//                            half-word;
//     [32 rows][2 x fp16]    scales of the tile's two blocks, row r at 1024 + 4 r.
//   Q8 tile = 32 weights per row (one block), 1088 bytes:
//     [32 rows][32 B codes]  byte i = q_i ^ 0x80 (offset binary), k ascending;
//     [32 rows][fp16]        scale, row r at 1024 + 2 r.
//
// Every lane's code load is one 32-byte access and a warp's 32 loads cover
// 1024 consecutive bytes.  packed_bytes == canonical_bytes.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/qmm.h"

namespace qmm {

constexpr int kRowsPerGroup = 32;
constexpr int kQ4TileK = 64;
constexpr int kQ8TileK = 32;
constexpr int kQ4TileBytes = 1152;
constexpr int kQ8TileBytes = 1088;
constexpr int kTileCodeBytes = 1024;
constexpr int kNumSMs = 148;

//   Q5 / Q6 tile = 64 weights per row, as Q4 plus a plane of high bits between codes and scales:
//     [32 rows][32 B low nibbles]  exactly the Q4 code layout, holding u & 15 (u = q + 16 / q + 32);
//     [32 rows][8 B] (Q5) / [32 rows][16 B] (Q6)  high bits.  Q5: two 32-bit words per row, word b for the
//                            packed words 4b .. 4b+3; the pair p of packed word j (elements 8j+2p, 8j+2p+1)
//                            has its fifth bits at bit t = 4 (j mod 4) + p and 16 + t, so one shift and a
//                            mask 0x00010001 << s drops them beside the low nibbles of both half-words.
//                            Q6: four words per row, word h for the packed words 2h, 2h+1; the pair's
//                            2-bit fields at bits 2t', 2t'+1 and 16 + 2t', t' = 4 (j mod 2) + p;
//     [32 rows][2 x fp16]    scales.                       Q5: 1408 bytes, Q6: 1664 bytes per tile.
constexpr int kQ5TileBytes = 1408;
constexpr int kQ6TileBytes = 1664;

template <int FMT> struct Fmt;
template <> struct Fmt<QMM_Q4> {
    static constexpr int tile_k = kQ4TileK;
    static constexpr int tile_bytes = kQ4TileBytes;
    static constexpr int canon_block = 18;
    static constexpr int hi_bytes = 0;                       // bytes of high bits per row and tile
    static constexpr int scale_off = kTileCodeBytes;         // offset of the scale plane in a tile
};
template <> struct Fmt<QMM_Q5> {
    static constexpr int tile_k = 64;
    static constexpr int tile_bytes = kQ5TileBytes;
    static constexpr int canon_block = 22;
    static constexpr int hi_bytes = 8;
    static constexpr int scale_off = kTileCodeBytes + 32 * 8;
};
template <> struct Fmt<QMM_Q6> {
    static constexpr int tile_k = 64;
    static constexpr int tile_bytes = kQ6TileBytes;
    static constexpr int canon_block = 26;
    static constexpr int hi_bytes = 16;
    static constexpr int scale_off = kTileCodeBytes + 32 * 16;
};
template <> struct Fmt<QMM_Q8> {
    static constexpr int tile_k = kQ8TileK;
    static constexpr int tile_bytes = kQ8TileBytes;
    static constexpr int canon_block = 34;
    static constexpr int hi_bytes = 0;
    static constexpr int scale_off = kTileCodeBytes;
};

__host__ __device__ inline int tile_k_of(int fmt) { return fmt == QMM_Q8 ? kQ8TileK : 64; }
__host__ __device__ inline int tile_bytes_of(int fmt)
{
    return fmt == QMM_Q4 ? kQ4TileBytes : fmt == QMM_Q5 ? kQ5TileBytes : fmt == QMM_Q6 ? kQ6TileBytes : kQ8TileBytes;
}
__host__ __device__ inline int canon_block_of(int fmt) { return fmt == QMM_Q4 ? 18 : fmt == QMM_Q5 ? 22 : fmt == QMM_Q6 ? 26 : 34; }

// Host-side error reporting (thread-local buffer; see qmm_api.cu).
qmm_status fail(qmm_status code, const char* fmt, ...);
qmm_status check_cuda(cudaError_t e, const char* what);

// Debug knobs set through qmm_debug_config (tests and tuning sweeps force launch geometries
// with them; none changes a result beyond the order of fp32 additions).  Plain process-wide
// values, all zero by default: the launch path reads them and nothing else -- no environment
// variable is looked at after the library is loaded.
struct DebugKnobs {
    int gemv_warps, gemv_splits;    // 0: the plan decides
    int gemv_no_cluster;            // split-K GEMV through workspace partial sums and a second kernel
    int gemm_bn, gemm_units;        // token tile / (tile, k-block) units per block of the dense GEMM; 0: the plan decides
    int gemm_no_tail_cut;           // leave the tiles of the last, partly filled round whole
    int gemm_no_small;              // M <= 8 through the tensor-core prefill kernel instead of the few-token kernel
    int moe_no_fuse;                // decode-sized MoE layers as four separate launches
};
extern DebugKnobs g_knobs;

// Arguments of the decode-sized mixture-of-experts layer (host side; see moe_small_gate_up_kernel).
struct MoeSmallHost {
    const float* logits; const uint16_t* X; const void *w_gate, *w_up, *w_down; int64_t gu_stride, dn_stride;
    uint16_t *hbuf, *dbg_D, *out; int T, E, topk, H, I;
    int* idx_ws; float* w_ws; int *perm_ws, *inv_ws, *offsets_ws;
    int* idx_user; float* w_user; int *perm_user, *offsets_user;
    long long* trace;           // tuning builds only, else null
};


// ---------------------------------------------------------------- loads

struct __align__(32) u32x8 {
    uint32_t v[8];
};

// 32-byte streaming load of weight codes: read-only path, no L1 allocation,
// first in line for L2 eviction (each byte is used once per product).
__device__ __forceinline__ u32x8 ld_stream_256(const void* p)
{
    u32x8 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::evict_first.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]),
                   "=r"(r.v[4]), "=r"(r.v[5]), "=r"(r.v[6]), "=r"(r.v[7])
                 : "l"(p));
    return r;
}

// Same bytes, but kept in L2 (weights that are re-read by other thread blocks).
__device__ __forceinline__ u32x8 ld_keep_256(const void* p)
{
    u32x8 r;
    asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]),
                   "=r"(r.v[4]), "=r"(r.v[5]), "=r"(r.v[6]), "=r"(r.v[7])
                 : "l"(p));
    return r;
}

__device__ __forceinline__ uint32_t ld_nc_u32(const void* p)
{
    uint32_t r;
    asm volatile("ld.global.nc.u32 %0, [%1];" : "=r"(r) : "l"(p));
    return r;
}

__device__ __forceinline__ uint16_t ld_nc_u16(const void* p)
{
    uint16_t r;
    asm volatile("ld.global.nc.u16 %0, [%1];" : "=h"(r) : "l"(p));
    return r;
}

// ------------------------------------------------ integer codes -> fp16

__device__ __forceinline__ __half2 as_h2(uint32_t u)
{
    return *reinterpret_cast<__half2*>(&u);
}
__device__ __forceinline__ uint32_t as_u32(__half2 h)
{
    return *reinterpret_cast<uint32_t*>(&h);
}

// Bit constants of the Q4 unpack, held in registers.  (a & mask) | magic is one
// LOP3 only when at most one of its operands is an immediate, so the values
// are produced by opaque moves that the compiler cannot fold back into
// immediates.
struct Q4Consts {
    uint32_t mask_lo, mask_hi, magic;
    __device__ __forceinline__ void init()
    {
        asm volatile("mov.u32 %0, 0x000F000F;" : "=r"(mask_lo));
        asm volatile("mov.u32 %0, 0x00F000F0;" : "=r"(mask_hi));
        asm volatile("mov.u32 %0, 0x64006400;" : "=r"(magic));
    }
};

__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c)
{
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));   // (a & b) | c
    return d;
}

// Q4: the four element pairs of one packed word as exact integers q in fp16.
// 0x6400 | u is the fp16 value 1024 + u; 0x6400 | (u << 4) is 1024 + 16 u.
// (1024 + u) - 1032 = q and (1024 + 16 u) / 16 - 72 = q are both exact.
__device__ __forceinline__ void q4_word_to_h2(uint32_t w, __half2 (&q)[4], const Q4Consts& k)
{
    const __half2 c1032 = as_h2(0x64086408u);
    const __half2 c16th = as_h2(0x2C002C00u);
    const __half2 cm72 = as_h2(0xD480D480u);
    const uint32_t w8 = w >> 8;
    q[0] = __hsub2(as_h2(and_or(w, k.mask_lo, k.magic)), c1032);
    q[1] = __hfma2(as_h2(and_or(w, k.mask_hi, k.magic)), c16th, cm72);
    q[2] = __hsub2(as_h2(and_or(w8, k.mask_lo, k.magic)), c1032);
    q[3] = __hfma2(as_h2(and_or(w8, k.mask_hi, k.magic)), c16th, cm72);
}

// Q5 / Q6: the four element pairs of packed word `j` of a tile as exact integers q in fp16.  `H` is the
// high-bit word that covers word j (see the layout above); the pair's high bits are shifted beside
// its low nibbles -- bit 4 (5) for the pairs taken with mask_lo, bit 8 (9) for those taken with mask_hi,
// whose value is then divided by 16 like the nibble -- and merged with one more LOP3.
// 0x6400 | u is 1024 + u: (1024 + u) - (1024 + OFF) = q, (1024 + 16 u) / 16 - (64 + OFF) = q, OFF = 16 / 32.
template <int FMT>
__device__ __forceinline__ void q56_word_to_h2(uint32_t w, uint32_t H, int j, __half2 (&q)[4], const Q4Consts& k)
{
    constexpr bool Q5 = FMT == QMM_Q5;
    const __half2 c_lo = as_h2(Q5 ? 0x64106410u : 0x64206420u);          // 1040 / 1056
    const __half2 c16th = as_h2(0x2C002C00u);
    const __half2 c_hi = as_h2(Q5 ? 0xD500D500u : 0xD600D600u);          // -80 / -96
    const uint32_t m_lo = Q5 ? 0x00100010u : 0x00300030u, m_hi = Q5 ? 0x01000100u : 0x03000300u;
    const uint32_t w8 = w >> 8;
    auto hi_at = [&](int p, int target) -> uint32_t {                      // the pair's high bits moved to bit `target`
        const int from = Q5 ? 4 * (j & 3) + p : 2 * (4 * (j & 1) + p);
        const int s = from - target;                                       // a constant once the callers' loops are unrolled
        return s >= 0 ? H >> s : H << -s;
    };
    q[0] = __hsub2(as_h2(and_or(hi_at(0, 4), m_lo, and_or(w, k.mask_lo, k.magic))), c_lo);
    q[1] = __hfma2(as_h2(and_or(hi_at(1, 8), m_hi, and_or(w, k.mask_hi, k.magic))), c16th, c_hi);
    q[2] = __hsub2(as_h2(and_or(hi_at(2, 4), m_lo, and_or(w8, k.mask_lo, k.magic))), c_lo);
    q[3] = __hfma2(as_h2(and_or(hi_at(3, 8), m_hi, and_or(w8, k.mask_hi, k.magic))), c16th, c_hi);
}

// Q8: the two element pairs of one packed word (4 offset-binary bytes) as
// exact integers in fp16.  0x6400 | (q + 128) is 1024 + 128 + q.
__device__ __forceinline__ void q8_word_to_h2(uint32_t w, __half2 (&q)[2])
{
    const __half2 c1152 = as_h2(0x64806480u);
    q[0] = __hsub2(as_h2(__byte_perm(w, 0x64646464u, 0x4140)), c1152);
    q[1] = __hsub2(as_h2(__byte_perm(w, 0x64646464u, 0x4342)), c1152);
}

// Programmatic dependent launch: let the next kernel in the stream start its
// prologue now / wait until the previous kernel's writes are visible.
__device__ __forceinline__ void pdl_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;");
}
__device__ __forceinline__ void pdl_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace qmm
