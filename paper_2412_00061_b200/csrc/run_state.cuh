// Running soft-max / top-k state shared by the draft-head kernels.
#pragma once

#include "common.cuh"

#include <limits.h>
#include <math.h>

namespace ctcsd {

// Running state for one (activation row, slot): online log-sum-exp plus the best 8 logits.
struct RunState {
    float mx, sum;
    float val[kTopSlots];
    int id[kTopSlots];

    __device__ __forceinline__ void init() {
        mx = -INFINITY;
        sum = 0.f;
#pragma unroll
        for (int s = 0; s < kTopSlots; ++s) { val[s] = -INFINITY; id[s] = INT_MAX; }
    }
    __device__ __forceinline__ void push(float z, int v) {
        if (z > mx) {
            sum = sum * __expf(mx - z) + 1.f;     // exp(-inf) = 0 covers the first element
            mx = z;
        } else {
            sum += __expf(z - mx);
        }
        topk_insert(val, id, z, v);
    }
    // push() keeping only the best KS logits
    template <int KS>
    __device__ __forceinline__ void push_n(float z, int v) {
        if (z > mx) {
            sum = sum * __expf(mx - z) + 1.f;
            mx = z;
        } else {
            sum += __expf(z - mx);
        }
        topk_insert_n<KS>(val, id, z, v);
    }
    __device__ __forceinline__ void absorb(const DraftPartial& q) {
        if (q.mx == -INFINITY) return;
        float nm = fmaxf(mx, q.mx);
        sum = (mx == -INFINITY ? 0.f : sum * __expf(mx - nm)) + q.sum * __expf(q.mx - nm);
        mx = nm;
#pragma unroll
        for (int s = 0; s < kTopSlots; ++s)
            if (q.id[s] != INT_MAX) topk_insert(val, id, q.val[s], q.id[s]);
    }
    __device__ __forceinline__ void store(DraftPartial* dst) const {
        dst->mx = mx;
        dst->sum = sum;
#pragma unroll
        for (int s = 0; s < kTopSlots; ++s) { dst->val[s] = val[s]; dst->id[s] = id[s]; }
    }
};

// Reads a partial that another CTA wrote (through L2, never a stale L1 line).
__device__ __forceinline__ DraftPartial load_partial_cg(const DraftPartial* src) {
    DraftPartial q;
    const int4* s4 = reinterpret_cast<const int4*>(src);
    int4* d4 = reinterpret_cast<int4*>(&q);
#pragma unroll
    for (int i = 0; i < (int)(sizeof(DraftPartial) / 16); ++i) d4[i] = __ldcg(s4 + i);
    return q;
}

// Combines the 32 lane-local states of a warp.  Every lane returns the merged max and sum;
// the merged best-8 list (descending) is returned in every lane's val/id.
__device__ __forceinline__ void warp_combine(RunState& st) {
    float gmx = warp_max(st.mx);
    float s = (st.mx == -INFINITY) ? 0.f : st.sum * __expf(st.mx - gmx);
    float gsum = warp_sum(s);
    float ov[kTopSlots];
    int oi[kTopSlots];
#pragma unroll
    for (int round = 0; round < kTopSlots; ++round) {
        float bv = st.val[0];
        int bi = st.id[0];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            float tv = __shfl_xor_sync(0xffffffffu, bv, o);
            int ti = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ranks_before(tv, ti, bv, bi)) { bv = tv; bi = ti; }
        }
        ov[round] = bv;
        oi[round] = bi;
        if (st.id[0] == bi && bi != INT_MAX) {       // this lane owned the winner: pop it
#pragma unroll
            for (int q = 0; q < kTopSlots - 1; ++q) { st.val[q] = st.val[q + 1]; st.id[q] = st.id[q + 1]; }
            st.val[kTopSlots - 1] = -INFINITY;
            st.id[kTopSlots - 1] = INT_MAX;
        }
    }
    st.mx = gmx;
    st.sum = gsum;
#pragma unroll
    for (int q = 0; q < kTopSlots; ++q) { st.val[q] = ov[q]; st.id[q] = oi[q]; }
}

}  // namespace ctcsd
