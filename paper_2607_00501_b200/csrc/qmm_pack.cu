// qmm_pack.cu -- canonical blocks <-> device layout.
//
// qmm_pack is the library's stand-in for the offline conversion of a
// checkpoint into the runtime's native weight format (Sec. 3, Sec. 4.1 of the
// paper): it runs once per weight and only moves integers and bits.
// qmm_dequant expands the device layout to fp32 for validation.
#include "qmm_common.cuh"

namespace qmm {

// One thread per (row, tile).  Canonical blocks are 18 / 34 bytes, so they are
// read byte by byte; this kernel is not on the hot path.
template <int FMT>
__global__ void pack_kernel(const uint8_t* __restrict__ canon, uint8_t* __restrict__ packed,
                            int64_t N, int64_t tiles_per_row)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * tiles_per_row) return;
    const int64_t n = idx / tiles_per_row;
    const int64_t t = idx % tiles_per_row;
    const int64_t rg = n / kRowsPerGroup;
    const int r = (int)(n % kRowsPerGroup);
    uint8_t* tile = packed + (rg * tiles_per_row + t) * Fmt<FMT>::tile_bytes;
    uint32_t words[8];
    if (FMT == QMM_Q4) {
        const uint8_t* b0 = canon + (n * tiles_per_row * 2 + t * 2) * 18;
        uint16_t d[2];
#pragma unroll
        for (int blk = 0; blk < 2; ++blk) {
            const uint8_t* b = b0 + blk * 18;
            d[blk] = (uint16_t)(b[0] | (b[1] << 8));
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t w = 0;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t byte = b[2 + 4 * j + c];      // elements 8j+2c (low), 8j+2c+1 (high)
                    w |= (byte & 0x0Fu) << (4 * c);
                    w |= (byte >> 4) << (16 + 4 * c);
                }
                words[blk * 4 + j] = w;
            }
        }
        *reinterpret_cast<uint32_t*>(tile + kTileCodeBytes + 4 * r) = (uint32_t)d[0] | ((uint32_t)d[1] << 16);
    } else {
        const uint8_t* b = canon + (n * tiles_per_row + t) * 34;
        const uint16_t d = (uint16_t)(b[0] | (b[1] << 8));
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            uint32_t w = 0;
#pragma unroll
            for (int c = 0; c < 4; ++c) w |= (uint32_t)(b[2 + 4 * j + c] ^ 0x80u) << (8 * c);
            words[j] = w;
        }
        *reinterpret_cast<uint16_t*>(tile + kTileCodeBytes + 2 * r) = d;
    }
    uint4* dst = reinterpret_cast<uint4*>(tile + 32 * r);
    dst[0] = make_uint4(words[0], words[1], words[2], words[3]);
    dst[1] = make_uint4(words[4], words[5], words[6], words[7]);
}

// One thread per (row, tile): w = float(d) * float(q), plain integer decode.
template <int FMT>
__global__ void dequant_kernel(const uint8_t* __restrict__ packed, float* __restrict__ w_out,
                               int64_t N, int64_t K, int64_t tiles_per_row)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * tiles_per_row) return;
    // consecutive threads take consecutive rows of one tile (coalesced code reads)
    const int64_t rg = idx / (tiles_per_row * kRowsPerGroup);
    const int64_t rem = idx % (tiles_per_row * kRowsPerGroup);
    const int64_t t = rem / kRowsPerGroup;
    const int r = (int)(rem % kRowsPerGroup);
    const int64_t n = rg * kRowsPerGroup + r;
    const uint8_t* tile = packed + (rg * tiles_per_row + t) * Fmt<FMT>::tile_bytes;
    const uint4* src = reinterpret_cast<const uint4*>(tile + 32 * r);
    const uint4 lo = src[0], hi = src[1];
    const uint32_t words[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
    float* out = w_out + n * K + t * Fmt<FMT>::tile_k;
    if (FMT == QMM_Q4) {
        const uint32_t dd = *reinterpret_cast<const uint32_t*>(tile + kTileCodeBytes + 4 * r);
        const float d0 = __half2float(__ushort_as_half((uint16_t)(dd & 0xFFFFu)));
        const float d1 = __half2float(__ushort_as_half((uint16_t)(dd >> 16)));
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const float d = j < 4 ? d0 : d1;
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                const int ue = (int)((words[j] >> (4 * p)) & 0xFu);        // element 2p
                const int uo = (int)((words[j] >> (16 + 4 * p)) & 0xFu);   // element 2p+1
                out[8 * j + 2 * p] = d * (float)(ue - 8);
                out[8 * j + 2 * p + 1] = d * (float)(uo - 8);
            }
        }
    } else {
        const float d = __half2float(__ushort_as_half(*reinterpret_cast<const uint16_t*>(tile + kTileCodeBytes + 2 * r)));
#pragma unroll
        for (int j = 0; j < 8; ++j) {
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int q = (int)((words[j] >> (8 * c)) & 0xFFu) - 128;
                out[4 * j + c] = d * (float)q;
            }
        }
    }
}

// Q5 / Q6.  One thread per (row, tile): the low nibbles go where Q4 puts its codes, the high bits
// into the row's high-bit words in the order the kernels' shift-and-mask unpack expects.
template <int FMT>
__global__ void pack56_kernel(const uint8_t* __restrict__ canon, uint8_t* __restrict__ packed,
                              int64_t N, int64_t tiles_per_row)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * tiles_per_row) return;
    constexpr int BB = Fmt<FMT>::canon_block;
    constexpr int NIB = FMT == QMM_Q5 ? 6 : 10;                  // offset of the low nibbles in a canonical block
    const int64_t n = idx / tiles_per_row, t = idx % tiles_per_row;
    const int64_t rg = n / kRowsPerGroup;
    const int r = (int)(n % kRowsPerGroup);
    uint8_t* tile = packed + (rg * tiles_per_row + t) * Fmt<FMT>::tile_bytes;
    uint32_t words[8], high[4] = {0u, 0u, 0u, 0u};
    uint16_t d[2];
    const uint8_t* b0 = canon + (n * tiles_per_row * 2 + t * 2) * BB;
    for (int blk = 0; blk < 2; ++blk) {
        const uint8_t* b = b0 + blk * BB;
        d[blk] = (uint16_t)(b[0] | (b[1] << 8));
        for (int j = 0; j < 4; ++j) {
            uint32_t w = 0;
            for (int c = 0; c < 4; ++c) {
                const uint32_t byte = b[NIB + 4 * j + c];         // elements 8j+2c (low nibble), 8j+2c+1 (high nibble)
                w |= (byte & 0x0Fu) << (4 * c);
                w |= (byte >> 4) << (16 + 4 * c);
            }
            words[blk * 4 + j] = w;
        }
        for (int i = 0; i < 32; ++i) {                           // element i of the block = element 32 blk + i of the tile
            const int j = 4 * blk + i / 8, pr = (i % 8) / 2, odd = i & 1;
            if (FMT == QMM_Q5) {
                const uint32_t bit = (b[2 + i / 8] >> (i % 8)) & 1u;
                high[blk] |= bit << (4 * (j & 3) + pr + 16 * odd);
            } else {
                const uint32_t two = (b[2 + i / 4] >> (2 * (i % 4))) & 3u;
                high[j / 2] |= two << (2 * (4 * (j & 1) + pr) + 16 * odd);
            }
        }
    }
    uint4* dst = reinterpret_cast<uint4*>(tile + 32 * r);
    dst[0] = make_uint4(words[0], words[1], words[2], words[3]);
    dst[1] = make_uint4(words[4], words[5], words[6], words[7]);
    uint32_t* hdst = reinterpret_cast<uint32_t*>(tile + kTileCodeBytes + Fmt<FMT>::hi_bytes * r);
    for (int i = 0; i < Fmt<FMT>::hi_bytes / 4; ++i) hdst[i] = high[i];
    *reinterpret_cast<uint32_t*>(tile + Fmt<FMT>::scale_off + 4 * r) = (uint32_t)d[0] | ((uint32_t)d[1] << 16);
}

// Q5 / Q6 device layout -> fp32, plain integer decode (validation).
template <int FMT>
__global__ void dequant56_kernel(const uint8_t* __restrict__ packed, float* __restrict__ w_out,
                                 int64_t N, int64_t K, int64_t tiles_per_row)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * tiles_per_row) return;
    const int64_t rg = idx / (tiles_per_row * kRowsPerGroup);
    const int64_t rem = idx % (tiles_per_row * kRowsPerGroup);
    const int64_t t = rem / kRowsPerGroup;
    const int r = (int)(rem % kRowsPerGroup);
    const int64_t n = rg * kRowsPerGroup + r;
    const uint8_t* tile = packed + (rg * tiles_per_row + t) * Fmt<FMT>::tile_bytes;
    const uint32_t* words = reinterpret_cast<const uint32_t*>(tile + 32 * r);
    const uint32_t* high = reinterpret_cast<const uint32_t*>(tile + kTileCodeBytes + Fmt<FMT>::hi_bytes * r);
    const uint32_t dd = *reinterpret_cast<const uint32_t*>(tile + Fmt<FMT>::scale_off + 4 * r);
    const float d0 = __half2float(__ushort_as_half((uint16_t)(dd & 0xFFFFu)));
    const float d1 = __half2float(__ushort_as_half((uint16_t)(dd >> 16)));
    float* out = w_out + n * K + t * 64;
    for (int j = 0; j < 8; ++j) {
        const float d = j < 4 ? d0 : d1;
        for (int e = 0; e < 8; ++e) {                            // element 8j + e: pair e / 2, low or high half-word
            const int pr = e / 2, odd = e & 1;
            const int lo = (int)((words[j] >> (4 * pr + 16 * odd)) & 0xFu);
            int u;
            if (FMT == QMM_Q5)
                u = lo | (int)(((high[j / 4] >> (4 * (j & 3) + pr + 16 * odd)) & 1u) << 4);
            else
                u = lo | (int)(((high[j / 2] >> (2 * (4 * (j & 1) + pr) + 16 * odd)) & 3u) << 4);
            out[8 * j + e] = d * (float)(u - (FMT == QMM_Q5 ? 16 : 32));
        }
    }
}

// Plausibility check of a packed buffer: one thread per (row, tile) looks at the row's scale(s) where
// the layout of `FMT` puts them.  A scale that is inf / NaN, or so large that |d| * max|q| leaves the
// fp16 range (the tensor-core products multiply d * q in fp16), marks the buffer as bad.  Bytes that are
// not a packed buffer of this format and shape (canonical blocks, the other format) put code bytes where
// scales are expected, and code bytes fail this test within a few hundred values.
template <int FMT>
__global__ void packed_check_kernel(const uint8_t* __restrict__ packed, int64_t N, int64_t tiles_per_row, int* __restrict__ status)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= N * tiles_per_row) return;
    const int64_t tile_idx = idx / kRowsPerGroup;                         // tiles are consecutive in memory
    const int r = (int)(idx % kRowsPerGroup);
    const uint8_t* tile = packed + tile_idx * Fmt<FMT>::tile_bytes;
    constexpr float kMaxAbs = 65504.0f / (FMT == QMM_Q4 ? 8.0f : FMT == QMM_Q5 ? 16.0f : FMT == QMM_Q6 ? 32.0f : 128.0f);
    bool bad = false;
    auto look = [&](uint16_t bits) {
        const float d = __half2float(__ushort_as_half(bits));
        bad |= !(fabsf(d) < kMaxAbs);                                     // also true for NaN
    };
    if (FMT != QMM_Q8) {
        const uint32_t dd = *reinterpret_cast<const uint32_t*>(tile + Fmt<FMT>::scale_off + 4 * r);
        look((uint16_t)(dd & 0xFFFFu));
        look((uint16_t)(dd >> 16));
    } else {
        look(*reinterpret_cast<const uint16_t*>(tile + kTileCodeBytes + 2 * r));
    }
    if (bad) atomicExch(status, (int)QMM_ERR_BAD_WEIGHTS);
}

qmm_status launch_packed_check(int fmt, const void* packed, int64_t N, int64_t K, int* status, cudaStream_t st)
{
    const int64_t tpr = K / tile_k_of(fmt);
    const int64_t total = N * tpr;
    const int threads = 256;
    const int64_t blocks = (total + threads - 1) / threads;
    if (fmt == QMM_Q4)
        packed_check_kernel<QMM_Q4><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)packed, N, tpr, status);
    else if (fmt == QMM_Q5)
        packed_check_kernel<QMM_Q5><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)packed, N, tpr, status);
    else if (fmt == QMM_Q6)
        packed_check_kernel<QMM_Q6><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)packed, N, tpr, status);
    else
        packed_check_kernel<QMM_Q8><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)packed, N, tpr, status);
    return check_cuda(cudaGetLastError(), "qmm_packed_check launch");
}

qmm_status launch_pack(int fmt, const void* canon, int64_t N, int64_t K, void* packed, cudaStream_t st)
{
    const int64_t tpr = K / tile_k_of(fmt);
    const int64_t total = N * tpr;
    const int threads = 256;
    const int64_t blocks = (total + threads - 1) / threads;
    if (fmt == QMM_Q4)
        pack_kernel<QMM_Q4><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)canon, (uint8_t*)packed, N, tpr);
    else if (fmt == QMM_Q5)
        pack56_kernel<QMM_Q5><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)canon, (uint8_t*)packed, N, tpr);
    else if (fmt == QMM_Q6)
        pack56_kernel<QMM_Q6><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)canon, (uint8_t*)packed, N, tpr);
    else
        pack_kernel<QMM_Q8><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)canon, (uint8_t*)packed, N, tpr);
    return check_cuda(cudaGetLastError(), "qmm_pack launch");
}

qmm_status launch_dequant(int fmt, const void* packed, int64_t N, int64_t K, float* w_out, cudaStream_t st)
{
    const int64_t tpr = K / tile_k_of(fmt);
    const int64_t total = N * tpr;
    const int threads = 256;
    const int64_t blocks = (total + threads - 1) / threads;
    if (fmt == QMM_Q4)
        dequant_kernel<QMM_Q4><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)packed, w_out, N, K, tpr);
    else if (fmt == QMM_Q5)
        dequant56_kernel<QMM_Q5><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)packed, w_out, N, K, tpr);
    else if (fmt == QMM_Q6)
        dequant56_kernel<QMM_Q6><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)packed, w_out, N, K, tpr);
    else
        dequant_kernel<QMM_Q8><<<(unsigned)blocks, threads, 0, st>>>((const uint8_t*)packed, w_out, N, K, tpr);
    return check_cuda(cudaGetLastError(), "qmm_dequant launch");
}

}  // namespace qmm
