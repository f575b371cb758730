// qmm_chain.cu -- a whole list of decode products, dependent or not, as ONE launch.
//
// The paper's decode argument (Sec. 3.3, Sec. 4.2): at one token per step every matrix-vector product
// is short, so what a runtime pays per product for dispatch and for the round trip between dependent
// kernels decides the token rate, and its answer is fused kernels and a low-overhead dispatch loop
// that is prepared once and replayed (Sec. 3.2).  The B200 counterpart built here: the products of a
// decode step (q/k/v, o, gate/up with SiLU*mul, down, layer after layer) are described once as a list
// of stages, a stage reading either a caller vector or the output of an earlier stage; a host-side
// planner turns the list into per-block work lists (`qmm_chain_build`, once); `qmm_chain_run` then is
// a single cooperative launch of one persistent block per SM.
//
// Inside a block
//   * a producer lane streams the block's weight tiles, in list order, into a shared-memory ring with
//     bulk asynchronous copies (cp.async.bulk, completion on an mbarrier).  Weights depend on nothing,
//     so the stream runs ahead of the dependency waits as far as the ring reaches: HBM keeps working
//     while a block waits for its activations;
//   * 16 consumer warps take one tile pair each per ring slot and multiply as the GEMV kernels do
//     (one matrix row per lane on the warp-level tensor path, qmm_gemv_core.cuh);
//   * a stage's outputs travel to their consumers as 32-bit words {fp16 value, 16-bit launch tag}:
//     one store publishes value and readiness together, a consumer block polls the words it needs and
//     no fence, counter or flag sits on the dependency path.  K splits (a stage too small to occupy
//     the SMs is cut along K) travel the same way as 64-bit words {fp32 partial sum, 32-bit tag}; the
//     block that owns a unit's last slice adds the slices in ascending order (a fixed order: same bits
//     on every call) and publishes the unit.
// Every wait (ring barriers, tag polls) is bounded; on give-up the block records
// QMM_ERR_DEVICE_TIMEOUT in the workspace's status word, which makes every other block stop as well.
#include "qmm_gemv_core.cuh"
#include "qmm_tc.cuh"

#include <algorithm>
#include <math.h>
#include <string.h>
#include <vector>

namespace qmm {

constexpr int kChainPairs = 16;                                 // tile pairs per ring slot
constexpr int kChainConsumers = 20;                             // consumer warps (16 of them work on any one slot)
constexpr int kChainPublishers = 2;                             // warps that reduce and publish a unit's 64 outputs
constexpr int kChainThreads = (kChainConsumers + 1 + kChainPublishers) * 32;   // + the producer warp
constexpr int kChainMaxSlices = 8;                              // K split of a stage: at most this many slices
constexpr int kChainMaxSlots = 6;
constexpr int kChainUnitCache = 160;                            // unit descriptors of a block kept in shared memory
constexpr int kChainMaxK = 32768;
constexpr uint32_t kChainMagic = 0x514D4348u;                   // "QMCH"
constexpr long long kChainWaitCycles = 1LL << 30;               // ~0.5 s: bound of every wait in the kernel

enum { kUnitPlain = 0, kUnitGateUp = 1 };
enum { kUnitNewX = 1 };

// One piece of work of a block: tiles [t0, t0 + nt) of a row-group pair (P, Q) of one stage.  All
// addresses are absolute device addresses (the plan is built for one workspace).
struct ChainUnit {
    const uint8_t* wp;          // tile t0 of row group P
    const uint8_t* wq;          // tile t0 of row group Q (next group of the matrix; the up matrix's group for gate/up)
    const uint8_t* x;           // the stage's activation vector: fp16 values, or tagged words {fp16, tag} (x_tagged)
    uint8_t* y_tag;             // tagged output words of this unit's first output
    uint16_t* y_plain;          // optional plain copy (this unit's first output), or null
    uint8_t* part;              // partial sums of the unit [nslices][64] words {fp32, tag} (nslices > 1)
    int32_t t0, nt;             // tile range along K
    int32_t kind;               // kUnitPlain: 64 outputs; kUnitGateUp: 32 outputs h = silu(g) * u
    int32_t slice, nslices;     // K split: this unit is slice `slice` of `nslices`
    int32_t flags;              // kUnitNewX: (re)stage the activation tiles [xt0, xt0 + xnt) before this unit
    int32_t xt0, xnt;
    int32_t x_tagged;           // != 0: x holds tagged words
    int32_t pad[3];
};
static_assert(sizeof(ChainUnit) == 96, "unit descriptor layout");

struct ChainHeader {            // start of the device plan buffer
    uint32_t magic;
    int32_t fmt, n_stages, n_units, grid, n_slots, max_k, pad;
    int64_t first_off, units_off;                               // byte offsets of the two arrays in the plan buffer
    const void* ws;                                             // the workspace the plan was built for
};

struct ChainCtl {               // start of the workspace
    int status;                 // 0, or a qmm_status recorded by a kernel (the status word of qmm_status_check)
    int pad;
    unsigned epoch;             // tag of the last completed launch
    unsigned exit_count;
};
constexpr size_t kChainCtlBytes = 256;

// ------------------------------------------------------------------ device

__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(tc::smem_u32(smem_dst)), "l"(gsrc), "r"(bytes), "r"(tc::smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ uint4 ld_volatile_v4(const void* p)
{
    uint4 v;
    asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint2 ld_volatile_v2(const void* p)        // one 64-bit word {value, tag}
{
    unsigned long long w;
    asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(w) : "l"(p) : "memory");
    return make_uint2((unsigned)w, (unsigned)(w >> 32));
}
__device__ __forceinline__ void st_word64(void* p, unsigned lo, unsigned hi)
{
    const unsigned long long w = (unsigned long long)lo | ((unsigned long long)hi << 32);
    asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(p), "l"(w) : "memory");
}
__device__ __forceinline__ void st_word32(void* p, unsigned w)
{
    asm volatile("st.volatile.global.u32 [%0], %1;" ::"l"(p), "r"(w) : "memory");
}
__device__ __forceinline__ int ld_volatile_int(const int* p)
{
    int v;
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Bounded wait that parks the warp instead of spinning: mbarrier.try_wait with a suspend-time hint
// lets the hardware hold the thread until the phase completes or the hint (in ns) has passed, so a
// waiting warp issues a handful of instructions per microsecond and leaves the issue slots to the
// warps that multiply.  Gives up like tc::mbar_wait: on the block's abort flag or after `limit` cycles.
__device__ __forceinline__ bool mbar_wait_parked(uint64_t* bar, uint32_t parity, volatile int* abort, long long limit)
{
    const uint32_t addr = tc::smem_u32(bar);
    const long long t0 = clock64();
    while (true) {
        uint32_t ok;
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t"
            "}\n"
            : "=r"(ok)
            : "r"(addr), "r"(parity), "r"(1000u)
            : "memory");
        if (ok) return true;
        if (*abort) return false;
        if (clock64() - t0 > limit) return false;
    }
}

__device__ __forceinline__ void consumer_sync()                       // the consumer warps only
{
    asm volatile("bar.sync 1, %0;" ::"r"(kChainConsumers * 32) : "memory");
}

// Barrier of the consumer warps that also tells whether every one of their threads is still fine.
__device__ __forceinline__ bool consumer_all(bool ok)
{
    uint32_t r;
    asm volatile(
        "{\n\t"
        ".reg .pred p, q;\n\t"
        "setp.ne.u32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}\n"
        : "=r"(r)
        : "r"((uint32_t)ok), "r"(kChainConsumers * 32)
        : "memory");
    return r != 0;
}

template <int FMT>
__global__ void __launch_bounds__(kChainThreads, 1)
chain_kernel(const uint8_t* __restrict__ plan, uint8_t* ws)
{
    using namespace tc;
    constexpr int TB = Fmt<FMT>::tile_bytes;
    constexpr int XV = Fmt<FMT>::tile_k / 8;                          // uint4 of activations per tile
    constexpr int SLOT = 2 * kChainPairs * TB;                        // bytes per ring slot: 16 tiles of P, 16 tiles of Q
    constexpr int NC = kChainConsumers;
    const ChainHeader* hd = reinterpret_cast<const ChainHeader*>(plan);
    const int* first = reinterpret_cast<const int*>(plan + hd->first_off);
    const ChainUnit* units = reinterpret_cast<const ChainUnit*>(plan + hd->units_off);
    ChainCtl* ctl = reinterpret_cast<ChainCtl*>(ws);
    const int NS = hd->n_slots;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    uint8_t* ring = smem;                                             // NS slots
    uint4* xs = reinterpret_cast<uint4*>(ring + (size_t)NS * SLOT);   // max_k fp16
    uint4* zs = xs + hd->max_k / 8;                                   // one tile of zeros
    float* red = reinterpret_cast<float*>(zs + XV);                   // [2][NC warps][64]: sums of a unit, double-buffered
    uint64_t* full = reinterpret_cast<uint64_t*>(red + 2 * NC * 64);  // [slots] copies landed
    uint64_t* empty = full + kChainMaxSlots;                          // [slots] consumers done
    uint64_t* red_full = empty + kChainMaxSlots;                      // [2] every consumer warp has written its sums
    uint64_t* red_empty = red_full + 2;                               // [2] the publishers have read them
    volatile int* s_abort = reinterpret_cast<volatile int*>(red_empty + 2);
    volatile unsigned* s_epoch = reinterpret_cast<volatile unsigned*>(s_abort + 1);
    ChainUnit* s_units = reinterpret_cast<ChainUnit*>(red_empty + 4); // [kChainUnitCache]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < kChainMaxSlots; ++s) {
            mbar_init(&full[s], 1);                                   // the producer's arrive (+ the copies' bytes)
            mbar_init(&empty[s], kChainPairs);                        // the 16 consumer warps that work on the slot
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&red_full[b], NC);
            mbar_init(&red_empty[b], kChainPublishers);
        }
        *s_abort = 0;
        // the tag of this launch: one more than the last completed launch's (all blocks read the same
        // value: it is only rewritten by the last block to leave, after every block has read it)
        *s_epoch = *reinterpret_cast<volatile unsigned*>(&ctl->epoch) + 1u;
        fence_barrier_init();
    }
    if (threadIdx.x < XV) zs[threadIdx.x] = make_uint4(0u, 0u, 0u, 0u);
    const int u_begin = first[blockIdx.x], u_end = first[blockIdx.x + 1];
    {
        // the block's unit descriptors (the first kChainUnitCache of them) into shared memory: a
        // descriptor read from global memory would be an L2 round trip on every dependent stage
        const int n16 = min(u_end - u_begin, kChainUnitCache) * (int)(sizeof(ChainUnit) / 16);
        const uint4* src = reinterpret_cast<const uint4*>(units + u_begin);
        for (int i = threadIdx.x; i < n16; i += kChainThreads) reinterpret_cast<uint4*>(s_units)[i] = src[i];
    }
    __syncthreads();
    const unsigned epoch = *s_epoch;
    const unsigned tag16 = epoch % 65535u + 1u;                       // 1 .. 65535; 0 = never written
    auto unit_at = [&](int ui) -> const ChainUnit* {
        return ui - u_begin < kChainUnitCache ? s_units + (ui - u_begin) : units + ui;
    };
    int polls = 0;
    // true while a poll of another block's data may go on: nobody has given up and the time limit holds
    auto may_wait = [&](long long t0) -> bool {
        if (*s_abort) return false;
        if ((++polls & 63) == 0) {
            if (ld_volatile_int(&ctl->status) != 0) return false;
            if (clock64() - t0 > kChainWaitCycles) return false;
        }
        return true;
    };
    bool gave_up = false;

    if (warp == NC) {
        // ================= producer: weight tiles -> ring, in list order, as far ahead as the ring reaches
        if (lane == 0) {
            int g = 0;
            bool ok = true;
            for (int ui = u_begin; ui < u_end && ok; ++ui) {
                const ChainUnit* up = unit_at(ui);
                const uint8_t* wp = up->wp;
                const uint8_t* wq = up->wq;
                const int nt = up->nt;
                for (int c = 0; c < nt && ok; c += kChainPairs, ++g) {
                    const int s = g % NS;
                    if (g >= NS) ok = mbar_wait_parked(&empty[s], ((g / NS) - 1) & 1, s_abort, kChainWaitCycles);
                    if (!ok) break;
                    const int np = min(kChainPairs, nt - c);
                    uint8_t* dst = ring + (size_t)s * SLOT;
                    mbar_arrive_expect_tx(&full[s], (uint32_t)(2 * np * TB));
                    bulk_g2s(dst, wp + (size_t)c * TB, (uint32_t)(np * TB), &full[s]);
                    bulk_g2s(dst + kChainPairs * TB, wq + (size_t)c * TB, (uint32_t)(np * TB), &full[s]);
                }
            }
            if (!ok) {
                gave_up = true;
                *s_abort = 1;
                // copies in flight must land before the block's shared memory is released
                for (int q = max(0, g - NS); q < g; ++q) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&full[q % NS], (q / NS) & 1) && clock64() - t0 < (1LL << 22)) {}
                }
            }
        }
    } else if (warp > NC) {
        // ================= publishers (64 threads): add the consumer warps' sums of a unit in warp order,
        // finish K splits, publish.  Decoupled from the consumers, which are already on the next unit.
        const int pt = threadIdx.x - (NC + 1) * 32;                   // output of the unit this thread owns
        bool ok = true;
        for (int ui = u_begin; ui < u_end && ok; ++ui) {
            const ChainUnit& u = *unit_at(ui);
            const int n = ui - u_begin, buf = n & 1;
            ok = mbar_wait_parked(&red_full[buf], (n >> 1) & 1, s_abort, kChainWaitCycles);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            const float* r = red + buf * (NC * 64);
            float v = 0.f;
            bool publish = true;
            if (u.kind == kUnitGateUp) {
                const int o = pt & 31;
                float gsum = r[o], usum = r[32 + o];
#pragma unroll
                for (int w = 1; w < NC; ++w) {
                    gsum += r[w * 64 + o];
                    usum += r[w * 64 + 32 + o];
                }
                v = (gsum / (1.0f + expf(-gsum))) * usum;
                publish = pt < 32;
            } else {
                v = r[pt];
#pragma unroll
                for (int w = 1; w < NC; ++w) v += r[w * 64 + pt];
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&red_empty[buf]);              // the consumers may reuse this buffer
            if (u.kind != kUnitGateUp && u.nslices > 1) {
                if (u.slice + 1 < u.nslices) {
                    st_word64(u.part + ((size_t)u.slice * 64 + pt) * 8, __float_as_uint(v), epoch);
                    publish = false;
                } else {
                    // the last slice adds the unit's slices in ascending order (its own last); all loads of
                    // a polling round are in flight together
                    const int others = u.nslices - 1;
                    uint2 w[kChainMaxSlices - 1];
                    const long long t0 = clock64();
#pragma unroll
                    for (int sl = 0; sl < kChainMaxSlices - 1; ++sl)
                        if (sl < others) w[sl] = ld_volatile_v2(u.part + ((size_t)sl * 64 + pt) * 8);
#pragma unroll
                    for (int sl = 0; sl < kChainMaxSlices - 1; ++sl) {
                        if (sl >= others || !ok) continue;
                        while (w[sl].y != epoch) {
                            if (!may_wait(t0)) {
                                ok = false;
                                break;
                            }
                            w[sl] = ld_volatile_v2(u.part + ((size_t)sl * 64 + pt) * 8);
                        }
                    }
                    float total = __uint_as_float(w[0].x);
#pragma unroll
                    for (int sl = 1; sl < kChainMaxSlices - 1; ++sl)
                        if (sl < others) total += __uint_as_float(w[sl].x);
                    v = total + v;
                }
            }
            if (publish && ok) {
                const unsigned hbits = __half_as_ushort(__float2half_rn(v));
                st_word32(u.y_tag + (size_t)pt * 4, hbits | (tag16 << 16));
                if (u.y_plain != nullptr) u.y_plain[pt] = (uint16_t)hbits;
            }
            ok = __all_sync(0xFFFFFFFFu, ok);
        }
        if (!ok) {
            gave_up = true;
            *s_abort = 1;
        }
    } else {
        // ================= consumers (NC warps).  A ring slot holds 16 tile pairs; the pairs of successive
        // slots go round the NC warps (pair i of slot g to warp (16 g + i) mod NC), so all of them work.
        const bool diag = (lane >> 2) == (lane & 3);
        const uint4* xbase = diag ? xs : zs;
        const int xmul = diag ? XV : 0;                               // off-diagonal lanes read the one tile of zeros
        Q4Consts kc;
        kc.init();
        int g = 0;
        int start = 0;                                                // (16 g) mod NC: the warp that takes pair 0 of slot g
        bool ok = true;
        // Control flow: every consumer thread passes the same sequence of consumer barriers (they only
        // surround the staging of an activation vector).  A thread that gives up raises the abort flag
        // (which ends every other wait of the block at once) and walks on without working; the vote at
        // the next staging barrier takes all of them out together.
        for (int ui = u_begin; ui < u_end; ++ui) {
            const ChainUnit& u = *unit_at(ui);
            const int n = ui - u_begin, buf = n & 1;
            if (u.flags & kUnitNewX) {
                consumer_sync();                                      // every warp is done with the previous vector
                const int v0 = u.xt0 * XV, v1 = (u.xt0 + u.xnt) * XV; // uint4 range of xs (8 fp16 each)
                if (!u.x_tagged) {
                    for (int i = v0 + (int)threadIdx.x; i < v1; i += NC * 32)
                        xs[i] = __ldcg(reinterpret_cast<const uint4*>(u.x) + i);
                } else if (ok) {
                    // tagged words {fp16, tag}: 8 values = two 16-byte loads; poll until every tag is this launch's
                    const long long t0 = clock64();
                    const unsigned want = tag16 << 16, m = 0xFFFF0000u;
                    for (int i0 = v0; i0 < v1 && ok; i0 += 2 * NC * 32) {
                        uint4 a[2], b[2];
#pragma unroll
                        for (int q = 0; q < 2; ++q) {                 // all loads of the round in flight at once
                            const int i = i0 + q * NC * 32 + (int)threadIdx.x;
                            if (i < v1) {
                                a[q] = ld_volatile_v4(u.x + (size_t)i * 32);
                                b[q] = ld_volatile_v4(u.x + (size_t)i * 32 + 16);
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            const int i = i0 + q * NC * 32 + (int)threadIdx.x;
                            if (i >= v1 || !ok) continue;
                            while (true) {
                                const bool have = ((a[q].x & m) == want) && ((a[q].y & m) == want) && ((a[q].z & m) == want) &&
                                                  ((a[q].w & m) == want) && ((b[q].x & m) == want) && ((b[q].y & m) == want) &&
                                                  ((b[q].z & m) == want) && ((b[q].w & m) == want);
                                if (have) break;
                                if (!may_wait(t0)) {
                                    ok = false;
                                    break;
                                }
                                a[q] = ld_volatile_v4(u.x + (size_t)i * 32);
                                b[q] = ld_volatile_v4(u.x + (size_t)i * 32 + 16);
                            }
                            if (ok)
                                xs[i] = make_uint4(__byte_perm(a[q].x, a[q].y, 0x5410), __byte_perm(a[q].z, a[q].w, 0x5410),
                                                   __byte_perm(b[q].x, b[q].y, 0x5410), __byte_perm(b[q].z, b[q].w, 0x5410));
                        }
                    }
                    if (!ok) *s_abort = 1;
                }
                ok = consumer_all(ok);                                // the vector is staged (or everyone leaves)
                if (!ok) break;
            }
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            const int nt = u.nt, t0u = u.t0;
            for (int c = 0; c < nt; c += kChainPairs, ++g) {
                int pi = warp - start;                                // this warp's pair of slot g, if < 16
                if (pi < 0) pi += NC;
                start += kChainPairs;
                if (start >= NC) start -= NC;
                if (!ok || pi >= kChainPairs) continue;
                const int s = g % NS;
                ok = mbar_wait_parked(&full[s], (g / NS) & 1, s_abort, kChainWaitCycles);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) {
                    *s_abort = 1;
                    continue;
                }
                if (c + pi < nt) {
                    const uint8_t* tp = ring + (size_t)s * SLOT + (size_t)pi * TB;
                    const uint8_t* tq = tp + kChainPairs * TB;
                    // the two 16-byte halves in an order that keeps a quarter-warp's accesses on distinct banks
                    const int h = (lane >> 2) & 1;
                    u32x8 cp, cq;
                    {
                        const uint4 p0 = *reinterpret_cast<const uint4*>(tp + 32 * lane + 16 * h);
                        const uint4 p1 = *reinterpret_cast<const uint4*>(tp + 32 * lane + 16 * (h ^ 1));
                        const uint4 q0 = *reinterpret_cast<const uint4*>(tq + 32 * lane + 16 * h);
                        const uint4 q1 = *reinterpret_cast<const uint4*>(tq + 32 * lane + 16 * (h ^ 1));
                        const uint4 plo = h ? p1 : p0, phi = h ? p0 : p1, qlo = h ? q1 : q0, qhi = h ? q0 : q1;
                        cp.v[0] = plo.x; cp.v[1] = plo.y; cp.v[2] = plo.z; cp.v[3] = plo.w;
                        cp.v[4] = phi.x; cp.v[5] = phi.y; cp.v[6] = phi.z; cp.v[7] = phi.w;
                        cq.v[0] = qlo.x; cq.v[1] = qlo.y; cq.v[2] = qlo.z; cq.v[3] = qlo.w;
                        cq.v[4] = qhi.x; cq.v[5] = qhi.y; cq.v[6] = qhi.z; cq.v[7] = qhi.w;
                    }
                    const int row = (lane & ~3) + 2 * (lane & 1);     // the rows whose sums this lane receives
                    const uint4* xt = xbase + (t0u + c + pi) * xmul;
                    if constexpr (FMT == QMM_Q4) {
                        const uint2 sp = *reinterpret_cast<const uint2*>(tp + kTileCodeBytes + 4 * row);
                        const uint2 sq = *reinterpret_cast<const uint2*>(tq + kTileCodeBytes + 4 * row);
                        tile_pair_mma_q4(cp, cq, sp, sq, xt, acc, kc);
                    } else {
                        const uint32_t sp = *reinterpret_cast<const uint32_t*>(tp + kTileCodeBytes + 2 * row);
                        const uint32_t sq = *reinterpret_cast<const uint32_t*>(tq + kTileCodeBytes + 2 * row);
                        tile_pair_mma_q8(cp, cq, sp, sq, xt, acc);
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&empty[s]);                // this warp is done with the slot
            }
            // hand the warp's sums to the publishers (buffer n & 1; its previous contents must have been read)
            if (ok && n >= 2) {
                ok = mbar_wait_parked(&red_empty[buf], ((n >> 1) - 1) & 1, s_abort, kChainWaitCycles);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) *s_abort = 1;
            }
            if (ok) {
                if ((lane & 3) < 2) {
                    const int row = (lane & ~3) + 2 * (lane & 1);
                    float* w = red + buf * (NC * 64) + warp * 64;
                    w[row] = acc[0];
                    w[row + 1] = acc[1];
                    w[32 + row] = acc[2];
                    w[32 + row + 1] = acc[3];
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&red_full[buf]);
            }
        }
        if (!ok) {
            gave_up = true;
            *s_abort = 1;
        }
    }

    // ---- leave: the last block to arrive records the launch's tag for the next launch
    if (gave_up) atomicExch(&ctl->status, (int)QMM_ERR_DEVICE_TIMEOUT);
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned old = atomicAdd(&ctl->exit_count, 1u);
        if (old == gridDim.x - 1) {
            ctl->exit_count = 0;
            __threadfence();
            *reinterpret_cast<volatile unsigned*>(&ctl->epoch) = epoch;
        }
    }
}

}  // namespace qmm

namespace qmm {

// ------------------------------------------------------------------ host: the planner

static size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct ChainLayout {
    std::vector<ChainUnit> units;       // grouped by block, in execution order; addresses relative (see place())
    std::vector<int> first;             // [grid + 1]
    std::vector<size_t> y_tag_off;      // per stage: byte offset of its tagged outputs in the workspace
    size_t ws_bytes = 0, plan_bytes = 0;
    int grid = kNumSMs, n_slots = 0, max_k = 0, smem_bytes = 0;
};

static qmm_status check_stages(const char* who, int fmt, const qmm_chain_stage* st, int count)
{
    if (fmt == QMM_Q5 || fmt == QMM_Q6) return fail(QMM_ERR_UNSUPPORTED, "%s: format %d is not built for this call", who, fmt);
    if (fmt != QMM_Q4 && fmt != QMM_Q8) return fail(QMM_ERR_INVALID_ARG, "%s: unknown format %d", who, fmt);
    if (!st || count <= 0) return fail(QMM_ERR_INVALID_ARG, "%s: empty stage list", who);
    if (count > 4096) return fail(QMM_ERR_UNSUPPORTED, "%s: %d stages > 4096", who, count);
    for (int i = 0; i < count; ++i) {
        const qmm_chain_stage& s = st[i];
        if (s.op != QMM_CHAIN_LINEAR && s.op != QMM_CHAIN_GATE_UP_SILU)
            return fail(QMM_ERR_INVALID_ARG, "%s: stage %d: unknown op %d", who, i, s.op);
        if (s.N <= 0 || s.K <= 0) return fail(QMM_ERR_INVALID_ARG, "%s: stage %d: N=%lld, K=%lld must be positive", who, i, (long long)s.N, (long long)s.K);
        if (s.K % 32) return fail(QMM_ERR_SHAPE, "%s: stage %d: K=%lld is not a multiple of the block size 32", who, i, (long long)s.K);
        if (s.K % 256 || s.N % 128 || s.K > kChainMaxK || s.N > (1 << 24))
            return fail(QMM_ERR_UNSUPPORTED, "%s: stage %d: needs K %% 256 == 0, N %% 128 == 0, K <= %d, N <= 2^24", who, i, kChainMaxK);
        if (!s.packed || (s.op == QMM_CHAIN_GATE_UP_SILU && !s.packed_up))
            return fail(QMM_ERR_INVALID_ARG, "%s: stage %d: null weight pointer", who, i);
        if ((reinterpret_cast<uintptr_t>(s.packed) & 31) || (reinterpret_cast<uintptr_t>(s.packed_up) & 31))
            return fail(QMM_ERR_ALIGNMENT, "%s: stage %d: packed weights must be 32-byte aligned", who, i);
        if (s.x_stage < 0) {
            if (!s.x_fp16) return fail(QMM_ERR_INVALID_ARG, "%s: stage %d: x_stage < 0 needs x_fp16", who, i);
            if (reinterpret_cast<uintptr_t>(s.x_fp16) & 15) return fail(QMM_ERR_ALIGNMENT, "%s: stage %d: x_fp16 must be 16-byte aligned", who, i);
        } else {
            if (s.x_stage >= i) return fail(QMM_ERR_SHAPE, "%s: stage %d reads stage %d, which is not an earlier stage", who, i, s.x_stage);
            if (s.x_offset < 0 || s.x_offset % 8 || s.x_offset + s.K > st[s.x_stage].N)
                return fail(QMM_ERR_SHAPE, "%s: stage %d: x_offset=%lld (a multiple of 8) + K=%lld must lie inside stage %d's %lld outputs",
                            who, i, (long long)s.x_offset, (long long)s.K, s.x_stage, (long long)st[s.x_stage].N);
        }
        if (reinterpret_cast<uintptr_t>(s.y_fp16) & 1) return fail(QMM_ERR_ALIGNMENT, "%s: stage %d: y_fp16 is misaligned", who, i);
    }
    return QMM_OK;
}

// Stage list -> per-block unit lists.  Stages whose inputs are ready together form a level (level 0:
// caller vectors; level l + 1: reads a stage of level l).  Within a level the units (64 output rows of a
// stage, or 32 gate/up outputs) are dealt to the blocks in list order in shares of equal bytes; a stage
// whose units alone cannot occupy its share of the blocks is cut along K into slices.  Units with earlier
// list positions never wait for later ones, and a block works through its list in order, so no wait
// can be circular.  Addresses in the units are offsets into the workspace where they point there
// (place() turns them into addresses).
static void plan_chain(int fmt, const qmm_chain_stage* st, int count, ChainLayout& L)
{
    const int TB = tile_bytes_of(fmt), TK = tile_k_of(fmt), G = kNumSMs;
    std::vector<int> level(count, 0);
    int n_levels = 0, max_k = 0;
    for (int i = 0; i < count; ++i) {
        level[i] = st[i].x_stage < 0 ? 0 : level[st[i].x_stage] + 1;
        n_levels = std::max(n_levels, level[i] + 1);
        max_k = std::max(max_k, (int)st[i].K);
    }
    // workspace: control words, tagged outputs of every stage, partial sums of split units
    size_t off = kChainCtlBytes;
    L.y_tag_off.assign(count, 0);
    for (int i = 0; i < count; ++i) {
        L.y_tag_off[i] = off;
        off = align_up(off + (size_t)st[i].N * 4, 256);
    }
    struct Item { ChainUnit u; int stage; long long cost; };
    std::vector<std::vector<ChainUnit>> per_block(G);
    for (int lv = 0; lv < n_levels; ++lv) {
        long long level_tiles = 0;
        for (int i = 0; i < count; ++i)
            if (level[i] == lv) level_tiles += (st[i].op == QMM_CHAIN_GATE_UP_SILU ? st[i].N / 32 : st[i].N / 64) * (st[i].K / TK);
        std::vector<Item> items;
        for (int i = 0; i < count; ++i) {
            if (level[i] != lv) continue;
            const qmm_chain_stage& s = st[i];
            const bool gu = s.op == QMM_CHAIN_GATE_UP_SILU;
            const int tpr = (int)(s.K / TK);
            const int n_units = (int)(gu ? s.N / 32 : s.N / 64);
            const size_t group_bytes = (size_t)tpr * TB;
            // K split: the slice count that minimises (rounds of this stage's items on its share of the blocks)
            // x (bytes of a slice), plus the price of the extra hop of the partial sums through L2 (measured: about
            // the time a block takes for 150 KB of weights, so only long-K stages with few rows are cut)
            int S = 1;
            if (!gu) {
                const double share = std::max(1.0, (double)G * ((double)n_units * tpr) / (double)std::max(1LL, level_tiles));
                double best = 1e30;
                for (int cand = 1; cand <= kChainMaxSlices; ++cand) {
                    const int per = (tpr + cand - 1) / cand;
                    if (cand > 1 && per < 4) break;
                    const double rounds = ceil((double)n_units * cand / share);
                    const double est = rounds * per * 2.0 * TB + (cand > 1 ? 150000.0 : 0.0);
                    if (est < best - 1e-9) {
                        best = est;
                        S = cand;
                    }
                }
            }
            for (int un = 0; un < n_units; ++un) {
                size_t part_off = 0;
                if (S > 1) {
                    part_off = off;
                    off += (size_t)S * 64 * 8;
                }
                for (int sl = 0; sl < S; ++sl) {
                    const int t0 = (int)((long long)tpr * sl / S), t1 = (int)((long long)tpr * (sl + 1) / S);
                    ChainUnit u;
                    memset(&u, 0, sizeof(u));
                    const uint8_t* w = (const uint8_t*)s.packed;
                    if (gu) {
                        u.wp = w + (size_t)un * group_bytes + (size_t)t0 * TB;
                        u.wq = (const uint8_t*)s.packed_up + (size_t)un * group_bytes + (size_t)t0 * TB;
                    } else {
                        u.wp = w + (size_t)(2 * un) * group_bytes + (size_t)t0 * TB;
                        u.wq = u.wp + group_bytes;
                    }
                    if (s.x_stage < 0) {
                        u.x = (const uint8_t*)s.x_fp16;
                        u.x_tagged = 0;
                    } else {
                        u.x = (const uint8_t*)(L.y_tag_off[s.x_stage] + (size_t)s.x_offset * 4);   // workspace offset
                        u.x_tagged = 1;
                    }
                    const int out0 = gu ? 32 * un : 64 * un;
                    u.y_tag = (uint8_t*)(L.y_tag_off[i] + (size_t)out0 * 4);                    // workspace offset
                    u.y_plain = s.y_fp16 ? s.y_fp16 + out0 : nullptr;
                    u.part = (uint8_t*)part_off;                                                // workspace offset
                    u.t0 = t0;
                    u.nt = t1 - t0;
                    u.kind = gu ? kUnitGateUp : kUnitPlain;
                    u.slice = sl;
                    u.nslices = S;
                    items.push_back({u, i, (long long)(t1 - t0)});
                }
            }
        }
        // Deal the items to the blocks.  Items that never wait for another block (whole units, and all
        // slices of a split unit but the last) come first in every block's list, the last slices (which
        // wait for the other slices of their unit) after them: when a block reaches one, the slices it
        // needs were started by their blocks at the same time as its own and are done or nearly so.
        // Many items: contiguous shares of equal cost (consecutive units of a stage stay together: one
        // staging of the activation vector).  Few items (a level of a dependent chain): each item to the
        // least loaded block, so that 128 items occupy 128 blocks.  The first block rotates with the level.
        const int rot = (int)(((long long)lv * 37) % G);
        std::vector<long long> load(G, 0);
        const bool contiguous = (long long)items.size() >= 4LL * G;
        for (int pass = 0; pass < 2; ++pass) {
            long long total = 0, before = 0;
            for (const Item& it : items)
                if ((it.u.nslices > 1 && it.u.slice + 1 == it.u.nslices) == (pass == 1)) total += it.cost;
            for (const Item& it : items) {
                if ((it.u.nslices > 1 && it.u.slice + 1 == it.u.nslices) != (pass == 1)) continue;
                int b;
                if (contiguous) {
                    const long long mid2 = 2 * before + it.cost;                // twice the item's midpoint
                    b = (int)((mid2 * G) / (2 * std::max(1LL, total)));
                    if (b >= G) b = G - 1;
                    before += it.cost;
                } else {
                    b = 0;
                    for (int k = 1; k < G; ++k)
                        if (load[k] < load[b]) b = k;
                }
                load[b] += it.cost;
                ChainUnit u = it.u;
                u.pad[0] = it.stage;                                            // (host only: which stage's vector the unit reads)
                per_block[(b + rot) % G].push_back(u);
            }
        }
    }
    off = align_up(off, 256);
    // activation staging: at a change of stage within a block, stage the tile range the run of units of that stage reads
    L.units.clear();
    L.first.assign(G + 1, 0);
    for (int b = 0; b < G; ++b) {
        std::vector<ChainUnit>& v = per_block[b];
        for (size_t i = 0; i < v.size();) {
            size_t j = i;
            int lo = v[i].t0, hi = v[i].t0 + v[i].nt;
            while (j + 1 < v.size() && v[j + 1].pad[0] == v[i].pad[0]) {
                ++j;
                lo = std::min(lo, v[j].t0);
                hi = std::max(hi, v[j].t0 + v[j].nt);
            }
            v[i].flags |= kUnitNewX;
            v[i].xt0 = lo;
            v[i].xnt = hi - lo;
            i = j + 1;
        }
        L.first[b] = (int)L.units.size();
        for (ChainUnit& u : v) {
            u.pad[0] = 0;
            L.units.push_back(u);
        }
    }
    L.first[G] = (int)L.units.size();
    L.ws_bytes = off;
    L.plan_bytes = align_up(sizeof(ChainHeader), 256) + align_up((size_t)(G + 1) * 4, 256) + L.units.size() * sizeof(ChainUnit);
    L.max_k = max_k;
    const int slot = 2 * kChainPairs * TB;
    const int fixed = 128 /*alignment*/ + max_k * 2 + (TK / 8) * 16 + 2 * kChainConsumers * 64 * 4 + (2 * kChainMaxSlots + 8) * 8 +
                      kChainUnitCache * (int)sizeof(ChainUnit) + 64;
    int ns = (227 * 1024 - fixed) / slot;
    L.n_slots = ns > kChainMaxSlots ? kChainMaxSlots : ns;
    L.smem_bytes = fixed + L.n_slots * slot;
}

size_t chain_plan_bytes(int fmt, const qmm_chain_stage* st, int count)
{
    if (check_stages("qmm_chain_plan_bytes", fmt, st, count) != QMM_OK) return 0;
    ChainLayout L;
    plan_chain(fmt, st, count, L);
    return L.plan_bytes;
}

size_t chain_workspace_bytes(int fmt, const qmm_chain_stage* st, int count)
{
    if (check_stages("qmm_chain_workspace_bytes", fmt, st, count) != QMM_OK) return 0;
    ChainLayout L;
    plan_chain(fmt, st, count, L);
    return L.ws_bytes;
}

qmm_status chain_build(int fmt, const qmm_chain_stage* st, int count, void* plan, size_t plan_bytes, void* ws, size_t ws_bytes,
                       qmm_chain_info* info, cudaStream_t stream)
{
    qmm_status s = check_stages("qmm_chain_build", fmt, st, count);
    if (s != QMM_OK) return s;
    if (!plan || !ws || !info) return fail(QMM_ERR_INVALID_ARG, "qmm_chain_build: null pointer");
    if ((reinterpret_cast<uintptr_t>(plan) & 255) || (reinterpret_cast<uintptr_t>(ws) & 255))
        return fail(QMM_ERR_ALIGNMENT, "qmm_chain_build: plan and workspace must be 256-byte aligned");
    ChainLayout L;
    plan_chain(fmt, st, count, L);
    if (plan_bytes < L.plan_bytes) return fail(QMM_ERR_WORKSPACE, "qmm_chain_build: plan buffer of %zu bytes needed, %zu given", L.plan_bytes, plan_bytes);
    if (ws_bytes < L.ws_bytes) return fail(QMM_ERR_WORKSPACE, "qmm_chain_build: workspace of %zu bytes needed, %zu given", L.ws_bytes, ws_bytes);
    if (L.n_slots < 2) return fail(QMM_ERR_UNSUPPORTED, "qmm_chain_build: K=%d leaves no room for the weight ring", L.max_k);
    // offsets into the workspace -> addresses
    uint8_t* wsb = (uint8_t*)ws;
    for (ChainUnit& u : L.units) {
        if (u.x_tagged) u.x = wsb + (size_t)u.x;
        u.y_tag = wsb + (size_t)u.y_tag;
        u.part = u.nslices > 1 ? wsb + (size_t)u.part : nullptr;
    }
    std::vector<uint8_t> host(L.plan_bytes, 0);
    ChainHeader hd;
    memset(&hd, 0, sizeof(hd));
    hd.magic = kChainMagic;
    hd.fmt = fmt;
    hd.n_stages = count;
    hd.n_units = (int)L.units.size();
    hd.grid = L.grid;
    hd.n_slots = L.n_slots;
    hd.max_k = L.max_k;
    hd.first_off = (int64_t)align_up(sizeof(ChainHeader), 256);
    hd.units_off = hd.first_off + (int64_t)align_up((size_t)(L.grid + 1) * 4, 256);
    hd.ws = ws;
    memcpy(host.data(), &hd, sizeof(hd));
    memcpy(host.data() + hd.first_off, L.first.data(), L.first.size() * 4);
    if (!L.units.empty()) memcpy(host.data() + hd.units_off, L.units.data(), L.units.size() * sizeof(ChainUnit));
    cudaError_t e = cudaMemsetAsync(ws, 0, L.ws_bytes, stream);              // tags 0 = never written, epoch 0, status 0
    if (e == cudaSuccess) e = cudaMemcpyAsync(plan, host.data(), L.plan_bytes, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);                 // the host copy of the plan is released on return
    if (e != cudaSuccess) return check_cuda(e, "qmm_chain_build");
    info->magic = (int32_t)kChainMagic;
    info->fmt = fmt;
    info->stages = count;
    info->grid = L.grid;
    info->threads = kChainThreads;
    info->smem_bytes = L.smem_bytes;
    info->plan_bytes = L.plan_bytes;
    info->ws_bytes = L.ws_bytes;
    info->plan = plan;
    info->ws = ws;
    return QMM_OK;
}

qmm_status chain_run(const qmm_chain_info* info, cudaStream_t stream)
{
    if (!info || info->magic != (int32_t)kChainMagic) return fail(QMM_ERR_INVALID_ARG, "qmm_chain_run: info was not filled by qmm_chain_build");
    const void* kern = info->fmt == QMM_Q4 ? (const void*)chain_kernel<QMM_Q4> : (const void*)chain_kernel<QMM_Q8>;
    static thread_local int configured_dev[2] = {-1, -1};                     // the attribute is per device and per kernel
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return check_cuda(e, "qmm_chain_run");
    const int which = info->fmt == QMM_Q4 ? 0 : 1;
    if (configured_dev[which] != dev) {
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return check_cuda(e, "qmm_chain_run shared memory size");
        configured_dev[which] = dev;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)info->grid);
    cfg.blockDim = dim3((unsigned)info->threads);
    cfg.dynamicSmemBytes = (size_t)info->smem_bytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;                              // the blocks wait on one another: all must be resident
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const uint8_t* plan = (const uint8_t*)info->plan;
    uint8_t* ws = (uint8_t*)info->ws;
    void* args[2] = {(void*)&plan, (void*)&ws};
    e = cudaLaunchKernelExC(&cfg, kern, args);
    return check_cuda(e, "qmm_chain_run launch");
}

}  // namespace qmm
