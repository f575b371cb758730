// qmm_route.cuh -- top-k routing of one token by one warp, shared by the mixture-of-experts kernels.
#pragma once

#include <cuda_runtime.h>
#include <math.h>

namespace qmm {

// Routing of one token by one warp.  topk passes; each pass takes the largest
// remaining logit, equal logits going to the lower expert index.  The weights
// are the softmax over the selected logits in fp32.  On return lane j < topk
// holds the j-th selected expert and its weight.
//
// A pass is two warp-wide integer reductions (redux.sync) instead of a
// shuffle tree over (value, index) pairs: logits are mapped to 32-bit keys
// whose unsigned order is the order of the floats (-0.0 first made +0.0, so
// that the two zeros tie as the rule says), the warp takes the maximum key,
// then the minimum expert index among the lanes that hold it.
__device__ __forceinline__ unsigned route_key(float v)
{
    const unsigned u = __float_as_uint(v + 0.0f);         // -0.0 + 0.0 = +0.0
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);    // > 0 for every float, -inf included
}
__device__ __forceinline__ float route_unkey(unsigned k)
{
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

template <int MAX_PER_LANE>
__device__ __forceinline__ void route_token(const float* __restrict__ l, int E, int topk, int lane, int& sel_idx, float& sel_w)
{
    unsigned key[MAX_PER_LANE];                           // 0: no such expert, or already selected
#pragma unroll
    for (int i = 0; i < MAX_PER_LANE; ++i) {
        const int e = lane + 32 * i;
        key[i] = e < E ? route_key(l[e]) : 0u;
    }
    float sel_val = 0.f, lmax = 0.f, denom = 0.f;         // lane j keeps the j-th selected logit
    sel_idx = 0;
    for (int j = 0; j < topk; ++j) {
        unsigned best = 0u;                               // this lane's largest remaining key; lowest expert on ties
        int best_i = 0;
#pragma unroll
        for (int i = 0; i < MAX_PER_LANE; ++i)
            if (key[i] > best) {
                best = key[i];
                best_i = i;
            }
        const unsigned top = __reduce_max_sync(0xFFFFFFFFu, best);
        const int best_e = (int)__reduce_min_sync(0xFFFFFFFFu, best == top ? (unsigned)(lane + 32 * best_i) : 0x7FFFFFFFu);
        if ((best_e & 31) == lane) {
#pragma unroll
            for (int i = 0; i < MAX_PER_LANE; ++i)
                if (i == (best_e >> 5)) key[i] = 0u;      // (constant indices: the array stays in registers)
        }
        const float val = route_unkey(top);
        if (j == 0) lmax = val;
        if (lane == j) {
            sel_val = val;
            sel_idx = best_e;
        }
        denom += expf(val - lmax);                        // same value and order on every lane
    }
    sel_w = expf(sel_val - lmax) / denom;
}

}  // namespace qmm
