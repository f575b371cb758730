// qmm_route.cuh -- top-k routing of one token by one warp, shared by the mixture-of-experts kernels.
#pragma once

#include <cuda_runtime.h>
#include <math.h>

namespace qmm {

// Routing of one token by one warp.  topk passes; each pass takes the largest
// remaining logit, equal logits going to the lower expert index.  The weights
// are the softmax over the selected logits in fp32.  On return lane j < topk
// holds the j-th selected expert and its weight.
template <int MAX_PER_LANE>
__device__ __forceinline__ void route_token(const float* __restrict__ l, int E, int topk, int lane, int& sel_idx, float& sel_w)
{
    float v[MAX_PER_LANE];
#pragma unroll
    for (int i = 0; i < MAX_PER_LANE; ++i) {
        const int e = lane + 32 * i;
        v[i] = e < E ? l[e] : -INFINITY;
    }
    unsigned taken = 0;                                   // bit i: v[i] already selected
    float sel_val = 0.f, lmax = 0.f, denom = 0.f;         // lane j keeps the j-th selected logit
    sel_idx = 0;
    for (int j = 0; j < topk; ++j) {
        float best = -INFINITY;
        int best_e = 0x7FFFFFFF;
#pragma unroll
        for (int i = 0; i < MAX_PER_LANE; ++i) {
            const int e = lane + 32 * i;
            if (e < E && !((taken >> i) & 1u) && (v[i] > best || (v[i] == best && e < best_e))) {
                best = v[i];
                best_e = e;
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float ob = __shfl_xor_sync(0xFFFFFFFFu, best, off);
            const int oe = __shfl_xor_sync(0xFFFFFFFFu, best_e, off);
            if (ob > best || (ob == best && oe < best_e)) {
                best = ob;
                best_e = oe;
            }
        }
        if ((best_e & 31) == lane) taken |= 1u << (best_e >> 5);
        if (j == 0) lmax = best;
        if (lane == j) {
            sel_val = best;
            sel_idx = best_e;
        }
        denom += expf(best - lmax);                       // same value and order on every lane
    }
    sel_w = expf(sel_val - lmax) / denom;
}

}  // namespace qmm
