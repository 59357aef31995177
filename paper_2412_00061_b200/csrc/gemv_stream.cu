// Weight-streaming matrix-vector kernel (see gemv_stream.cuh).
#include "gemv_stream.cuh"
#include "tc_primitives.cuh"

#include <limits.h>
#include <math.h>

namespace ctcsd {

namespace {

constexpr int kWarps = 8;                     // consumer warps
constexpr int kThreads = (kWarps + 1) * 32;   // plus one producer warp
constexpr int kMaxSlots = 32;                 // ring slots

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

// Shared-memory bookkeeping of the weight ring.
struct __align__(8) RingShared {
    uint64_t full[kMaxSlots];     // the slot's weight rows have landed
    uint64_t empty[kMaxSlots];    // every consumer warp of the slot has read its row
    int abort_flag;
    int never_set;                // stays zero: lets a drain wait run to its time limit after an abort
    int is_last;
};

// One CTA per SM.  Warp 8 is the producer: it walks the CTA's contiguous range of weight rows
// and copies `G` rows (about 32 KB) per ring slot with the bulk-copy engine, as far ahead as
// the ring allows (about 190 KB in flight per SM).  Warps 0..7 are consumers: they form 8/G
// groups that take the slots in turn; within a group each warp owns one row of the slot,
// multiplies it with the activation rows held in shared memory, frees the slot and folds the
// logit into its lanes' running (max, sum of exp, best-8) states.
template <typename T, int MROWS>
__global__ void __launch_bounds__(kThreads, 1) gemv_stream_kernel(GemvParams p, int nslots, int G) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int row_bytes = p.H * (int)sizeof(T);
    const int nch = row_bytes / 16;                                  // 16-byte chunks per row
    const int slot_bytes = G * row_bytes;
    uint4* xs = reinterpret_cast<uint4*>(smem_raw);                  // [MROWS][nch]
    unsigned char* ring = smem_raw + (size_t)MROWS * row_bytes;      // [nslots][G][row_bytes]
    RingShared* sh = reinterpret_cast<RingShared*>(ring + (size_t)nslots * slot_bytes);
    __shared__ DraftPartial s_part[2][kWarps][MROWS];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int* abort_flag = &sh->abort_flag;

    if (tid == 0) {
        for (int s = 0; s < nslots; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], G); }
        sh->abort_flag = 0;
        sh->never_set = 0;
        sh->is_last = 0;
        tc::fence_barrier_init();
    }
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
    const int ntotal = (int)(r1 - r0);                               // rows of this CTA
    const int nfill = (ntotal + G - 1) / G;                          // ring fills of this CTA
    const int slot0 = (int)(r0 / rps);
    const long long seg_end = (long long)(slot0 + 1) * rps;          // first row of the next slot
    const int n_seg0 = (int)((r1 < seg_end ? r1 : seg_end) - r0);    // rows that belong to slot0
    const unsigned char* Wbase = reinterpret_cast<const unsigned char*>(p.W);

    if (warp == kWarps) {
        // ---------------- producer ----------------
        if (lane == 0) {
            const uint64_t policy = tc::policy_evict_first();
            bool ok = true;
            int j = 0;
            for (; j < nfill; ++j) {
                const int s = j % nslots;
                const uint32_t ph = (uint32_t)(j / nslots) & 1u;
                if (!tc::mbar_wait(&sh->empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                const int rows = (ntotal - j * G < G) ? ntotal - j * G : G;
                const uint32_t bytes = (uint32_t)rows * (uint32_t)row_bytes;
                // never hand the copy engine a range outside the weights or the ring
                const long long first = r0 + (long long)j * G;
                if (rows < 1 || first < 0 || first + rows > R || (bytes & 15u) != 0 || bytes > (uint32_t)slot_bytes ||
                    s >= nslots) {
                    report_error(p.status, CTCSD_ERR_INTERNAL, 12);
                    ok = false;
                    break;
                }
                tc::mbar_arrive_expect_tx(&sh->full[s], bytes);
                tc::bulk_load_1d(ring + (size_t)s * slot_bytes, Wbase + (size_t)first * row_bytes, bytes,
                                 &sh->full[s], policy);
            }
            if (!ok) {
                if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 10);
                *abort_flag = 1;
            }
            if (*abort_flag != 0) {
                // let copies that are still in flight land before the CTA gives its memory back
                for (int back = 1; back <= nslots && back <= j; ++back) {
                    const int q = j - back;
                    tc::mbar_wait(&sh->full[q % nslots], (uint32_t)(q / nslots) & 1u, &sh->never_set, 1ll << 24);
                }
            }
        }
    } else {
        // ---------------- consumers ----------------
        RunState st;
        st.init();
        int cur_seg = 0;
        bool ok = true;
        const int groups = kWarps / G;
        const int rin = warp % G;                       // this warp's row within a slot
        for (int j = warp / G; j < nfill; j += groups) {
            const int s = j % nslots;
            const uint32_t ph = (uint32_t)(j / nslots) & 1u;
            if (!tc::mbar_wait(&sh->full[s], ph, abort_flag)) { ok = false; break; }
            const int i = j * G + rin;                  // row of the CTA's range
            float acc[MROWS];
#pragma unroll
            for (int m = 0; m < MROWS; ++m) acc[m] = 0.f;
            if (i < ntotal) {
                const uint4* wrow = reinterpret_cast<const uint4*>(ring + (size_t)s * slot_bytes + (size_t)rin * row_bytes);
#pragma unroll 4
                for (int ch = lane; ch < nch; ch += 32) {
                    const uint4 w = wrow[ch];
#pragma unroll
                    for (int m = 0; m < MROWS; ++m) acc[m] = Elem<T>::dot(w, xs[m * nch + ch], acc[m]);
                }
            }
            // the accumulators depend on every load of the row: the slot can be refilled
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&sh->empty[s]);
            if (i >= ntotal) continue;
            const int seg = i >= n_seg0 ? 1 : 0;
            if (seg != cur_seg) {                       // this warp's rows now belong to the next slot
                if (lane < MROWS) st.store(&s_part[0][warp][lane]);
                st.init();
                cur_seg = 1;
            }
#pragma unroll
            for (int m = 0; m < MROWS; ++m) acc[m] = warp_sum(acc[m]);
            float z = 0.f;
#pragma unroll
            for (int m = 0; m < MROWS; ++m) if (lane == m) z = acc[m];
            if (lane < p.mcount) {
                const int slot = slot0 + seg;
                const int v = (int)(r0 + i - (long long)slot * rps);
                if (v == (int)rps - 1) z += bias;
                if (p.logits_dbg) p.logits_dbg[((size_t)(p.m0 + lane) * p.slots + slot) * rps + v] = z;
                st.push(z, v);
            }
        }
        if (!ok && lane == 0) {
            if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 11);
            *abort_flag = 1;
        }
        if (lane < MROWS) {
            if (cur_seg == 0) {
                st.store(&s_part[0][warp][lane]);
                st.init();
            }
            st.store(&s_part[1][warp][lane]);
        }
    }
    __syncthreads();

    // fold the 8 warps' states per segment: warp m merges activation row m's states, one per lane
    for (int seg = 0; seg < 2; ++seg) {
        if (warp < MROWS) {
            RunState ms;
            ms.init();
            if (lane < kWarps) ms.absorb(s_part[seg][lane][warp]);
            warp_combine(ms);
            if (lane == 0) ms.store(p.part + ((size_t)warp * p.grid + blockIdx.x) * 2 + seg);
        }
        if (tid == 0) {
            const int nrows = seg == 0 ? n_seg0 : ntotal - n_seg0;
            p.part_slot[blockIdx.x * 2 + seg] = (nrows > 0 && slot0 + seg < p.slots) ? slot0 + seg : -1;
        }
    }

    // the last CTA to arrive merges every CTA's partials into the final outputs
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        unsigned t = atomicAdd(p.counter, 1u);
        sh->is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!sh->is_last) return;
    __threadfence();

    const int ntask = p.mcount * p.slots;
    for (int task = warp; task < ntask; task += kThreads / 32) {
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
    const size_t row_bytes = (size_t)p.H * sizeof(T);
    const size_t budget = 200 * 1024;                          // dynamic shared memory per CTA
    const size_t fixed = (size_t)MROWS * row_bytes + sizeof(RingShared);
    // rows per ring slot: a power of two that divides the 8 consumer warps, about 32 KB per copy
    int G = 1;
    while (G < kWarps && (size_t)(2 * G) * row_bytes <= 32 * 1024) G *= 2;
    while (G > 1 && fixed + 3 * (size_t)G * row_bytes > budget) G /= 2;
    const size_t slot_bytes = (size_t)G * row_bytes;
    if (fixed + 2 * slot_bytes > budget) return CTCSD_ERR_UNSUPPORTED;
    long long nslots = (long long)((budget - fixed) / slot_bytes);
    if (nslots > kMaxSlots) nslots = kMaxSlots;
    const size_t smem = fixed + (size_t)nslots * slot_bytes;
    CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    long long R = (long long)p.slots * p.rows_per_slot;
    long long grid = h->num_sms;
    if (grid > R) grid = R;
    if (grid < p.slots) grid = p.slots;         // a CTA's range then touches at most two slots
    p.grid = (int)grid;
    kern<<<(unsigned)grid, kThreads, smem, stream>>>(p, (int)nslots, G);
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
    p.status = status_ptr(h);
    if (dtype == CTCSD_DTYPE_BF16) return launch_typed<__nv_bfloat16>(h, stream, M, p);
    return launch_typed<float>(h, stream, M, p);
}

}  // namespace ctcsd
