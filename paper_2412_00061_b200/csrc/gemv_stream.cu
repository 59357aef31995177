// Weight-streaming matrix-vector kernel (see gemv_stream.cuh).
#include "gemv_stream.cuh"

#include <limits.h>
#include <math.h>

namespace ctcsd {

namespace {

constexpr int kRW = 4;            // weight rows a warp carries through one sweep over H
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

template <typename T> struct Elem;

template <> struct Elem<float> {
    __device__ static __forceinline__ float dot(const uint4& w, const uint4& x, float acc) {
        acc = fmaf(__uint_as_float(w.x), __uint_as_float(x.x), acc);
        acc = fmaf(__uint_as_float(w.y), __uint_as_float(x.y), acc);
        acc = fmaf(__uint_as_float(w.z), __uint_as_float(x.z), acc);
        acc = fmaf(__uint_as_float(w.w), __uint_as_float(x.w), acc);
        return acc;
    }
};

template <> struct Elem<__nv_bfloat16> {
    __device__ static __forceinline__ float dot(const uint4& w, const uint4& x, float acc) {
        acc = fmaf(bf16lo(w.x), bf16lo(x.x), acc);
        acc = fmaf(bf16hi(w.x), bf16hi(x.x), acc);
        acc = fmaf(bf16lo(w.y), bf16lo(x.y), acc);
        acc = fmaf(bf16hi(w.y), bf16hi(x.y), acc);
        acc = fmaf(bf16lo(w.z), bf16lo(x.z), acc);
        acc = fmaf(bf16hi(w.z), bf16hi(x.z), acc);
        acc = fmaf(bf16lo(w.w), bf16lo(x.w), acc);
        acc = fmaf(bf16hi(w.w), bf16hi(x.w), acc);
        return acc;
    }
};

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

template <typename T, int MROWS>
__global__ void __launch_bounds__(kThreads) gemv_stream_kernel(GemvParams p) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint4* xs = reinterpret_cast<uint4*>(smem_raw);                 // [MROWS][nch]
    __shared__ DraftPartial s_part[kWarps][MROWS];
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nch = p.H * (int)sizeof(T) / 16;                      // 16-byte chunks per row

    for (int i = tid; i < MROWS * nch; i += kThreads) {
        int m = i / nch, ch = i - m * nch;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (m < p.mcount) v = reinterpret_cast<const uint4*>(p.x)[(size_t)(p.m0 + m) * nch + ch];
        xs[i] = v;
    }
    float bias = 0.f;
    if (lane < p.mcount && p.blank_bias != nullptr) {
        int row = p.m0 + lane;
        bias = p.blank_bias[p.row_seq ? p.row_seq[row] : row];
    }
    __syncthreads();

    const long long rps = p.rows_per_slot;
    const long long R = rps * p.slots;
    const long long r0 = R * blockIdx.x / gridDim.x;
    const long long r1 = R * (blockIdx.x + 1) / gridDim.x;
    const int slot0 = (int)(r0 / rps);
    const uint4* Wbase = reinterpret_cast<const uint4*>(p.W);
    const uint64_t policy = l2_policy_evict_first();

    for (int seg = 0; seg < 2; ++seg) {
        const int slot = slot0 + seg;
        long long a = seg == 0 ? r0 : (long long)(slot0 + 1) * rps;
        long long b = seg == 0 ? (r1 < (long long)(slot0 + 1) * rps ? r1 : (long long)(slot0 + 1) * rps) : r1;
        const int nrows = b > a ? (int)(b - a) : 0;
        const int v0 = (int)(a - (long long)slot * rps);            // first class id of the segment

        RunState st;
        st.init();
        const int ngroups = (nrows + kRW - 1) / kRW;
        for (int g = warp; g < ngroups; g += kWarps) {
            const uint4* wp[kRW];
#pragma unroll
            for (int r = 0; r < kRW; ++r) {
                int lr = g * kRW + r;
                if (lr >= nrows) lr = nrows - 1;                     // clamp: loaded again, result unused
                wp[r] = Wbase + (size_t)(a + lr) * nch;
            }
            float acc[kRW][MROWS];
#pragma unroll
            for (int r = 0; r < kRW; ++r)
#pragma unroll
                for (int m = 0; m < MROWS; ++m) acc[r][m] = 0.f;

#pragma unroll 2
            for (int ch = lane; ch < nch; ch += 32) {
                uint4 w[kRW];
#pragma unroll
                for (int r = 0; r < kRW; ++r) w[r] = ld_stream16(wp[r] + ch, policy);
#pragma unroll
                for (int m = 0; m < MROWS; ++m) {
                    uint4 xv = xs[m * nch + ch];
#pragma unroll
                    for (int r = 0; r < kRW; ++r) acc[r][m] = Elem<T>::dot(w[r], xv, acc[r][m]);
                }
            }
#pragma unroll
            for (int r = 0; r < kRW; ++r)
#pragma unroll
                for (int m = 0; m < MROWS; ++m) acc[r][m] = warp_sum(acc[r][m]);

#pragma unroll
            for (int r = 0; r < kRW; ++r) {
                int lr = g * kRW + r;
                if (lr < nrows) {
                    float z = 0.f;
#pragma unroll
                    for (int m = 0; m < MROWS; ++m) if (lane == m) z = acc[r][m];
                    if (lane < p.mcount) {
                        int v = v0 + lr;
                        if (v == (int)rps - 1) z += bias;
                        if (p.logits_dbg)
                            p.logits_dbg[((size_t)(p.m0 + lane) * p.slots + slot) * rps + v] = z;
                        st.push(z, v);
                    }
                }
            }
        }

        // fold the 8 warps' states: warp m merges row m's states, one per lane
        if (lane < MROWS) st.store(&s_part[warp][lane]);
        __syncthreads();
        if (warp < MROWS) {
            RunState ms;
            ms.init();
            if (lane < kWarps) ms.absorb(s_part[lane][warp]);
            warp_combine(ms);
            if (lane == 0) {
                DraftPartial* dst = p.part + ((size_t)warp * p.grid + blockIdx.x) * 2 + seg;
                ms.store(dst);
            }
        }
        if (tid == 0) p.part_slot[blockIdx.x * 2 + seg] = (nrows > 0 && slot < p.slots) ? slot : -1;
        __syncthreads();
    }

    // the last CTA to arrive merges every CTA's partials into the final outputs
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        unsigned t = atomicAdd(p.counter, 1u);
        s_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    const int ntask = p.mcount * p.slots;
    for (int task = warp; task < ntask; task += kWarps) {
        const int m = task / p.slots, slot = task - m * p.slots;
        RunState fs;
        fs.init();
        for (int e = lane; e < 2 * (int)gridDim.x; e += 32) {
            if (__ldcg(p.part_slot + e) == slot) {
                DraftPartial q = load_partial_cg(p.part + (size_t)m * p.grid * 2 + e);
                fs.absorb(q);
            }
        }
        warp_combine(fs);
        if (lane == 0) {
            const int row = p.m0 + m;
            if (p.mode == 0) {
                float lse = fs.mx + logf(fs.sum);
                p.out_lse[(size_t)row * p.slots + slot] = lse;
#pragma unroll
                for (int j = 0; j < kTopSlots; ++j) {
                    if (j < p.k) {
                        size_t o = ((size_t)row * p.slots + slot) * p.k + j;
                        p.out_topk_id[o] = fs.id[j];
                        p.out_topk_lp[o] = fs.val[j] - lse;
                    }
                }
            } else {
                p.out_argmax[row] = fs.id[0];
            }
        }
    }
    if (tid == 0) *p.counter = 0u;
}

template <typename T, int MROWS>
int launch_one(Handle* h, cudaStream_t stream, GemvParams& p) {
    auto kern = gemv_stream_kernel<T, MROWS>;
    size_t smem = (size_t)MROWS * p.H * sizeof(T);
    if (smem > 200 * 1024) return CTCSD_ERR_UNSUPPORTED;
    if (smem > 48 * 1024)
        CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int occ = 0;
    CTCSD_CUDA_CHECK(h, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, kThreads, smem));
    if (occ < 1) return CTCSD_ERR_UNSUPPORTED;
    if (occ > 8) occ = 8;
    long long R = (long long)p.slots * p.rows_per_slot;
    long long grid = (long long)h->num_sms * occ;
    if (grid > R) grid = R;
    if (grid < p.slots) grid = p.slots;         // a CTA's range then touches at most two slots
    p.grid = (int)grid;
    kern<<<(unsigned)grid, kThreads, smem, stream>>>(p);
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}

template <typename T>
int launch_typed(Handle* h, cudaStream_t stream, int M, GemvParams& p) {
    for (int m0 = 0; m0 < M; m0 += 4) {
        p.m0 = m0;
        p.mcount = (M - m0 < 4) ? (M - m0) : 4;
        int rc;
        if (p.mcount == 1) rc = launch_one<T, 1>(h, stream, p);
        else if (p.mcount == 2) rc = launch_one<T, 2>(h, stream, p);
        else rc = launch_one<T, 4>(h, stream, p);
        if (rc != CTCSD_OK) return rc;
    }
    return CTCSD_OK;
}

}  // namespace

int launch_gemv_stream(Handle* h, cudaStream_t stream, int dtype, int M, GemvParams p) {
    p.part = reinterpret_cast<DraftPartial*>(h->ws + h->lay.draft_part_off);
    p.part_slot = reinterpret_cast<int*>(h->ws + h->lay.part_slot_off);
    p.counter = counter_ptr(h);
    if (dtype == CTCSD_DTYPE_BF16) return launch_typed<__nv_bfloat16>(h, stream, M, p);
    return launch_typed<float>(h, stream, M, p);
}

}  // namespace ctcsd
