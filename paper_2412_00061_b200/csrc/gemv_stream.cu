// Weight-streaming matrix-vector kernel (see gemv_stream.cuh).
#include "gemv_stream.cuh"
#include "tc_primitives.cuh"
#include "run_state.cuh"

#include <limits.h>
#include <math.h>

namespace ctcsd {

namespace {

constexpr int kWarps = 8;                     // consumer warps
constexpr int kEpiWarps = 4;                  // warps that fold logits into the running states (bf16 path)
constexpr int kThreads = (kWarps + 1 + kEpiWarps) * 32;   // consumers, one producer warp, epilogue warps
constexpr int kCDepth = 4;                    // partial-sum buffers between consumers and epilogue
constexpr int kMaxSlots = 32;                 // ring slots
constexpr int kRowsPerWarp = 2;               // a slot holds at most kWarps * kRowsPerWarp weight rows

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

// Shared-memory bookkeeping of the weight ring.
struct __align__(8) RingShared {
    uint64_t full[kMaxSlots];     // the slot's weight rows have landed
    uint64_t empty[kMaxSlots];    // every consumer warp has read its part of the slot
    uint64_t cfull[kCDepth];      // every consumer warp has written its partial sums of a fill
    uint64_t cempty[kCDepth];     // every epilogue warp has read them
    int abort_flag;
    int never_set;                // stays zero: lets a drain wait run to its time limit after an abort
    int is_last;
};

constexpr int kStateRows = 16;    // running states per activation row inside a CTA (merged at the end)

// D[16x8] += A[16x16] * B[16x8], bf16 operands, fp32 accumulators (warp-wide).
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                          uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <typename T> __device__ __forceinline__ void store_as(void* dst, size_t i, float v);
template <> __device__ __forceinline__ void store_as<float>(void* dst, size_t i, float v) { static_cast<float*>(dst)[i] = v; }
template <> __device__ __forceinline__ void store_as<__nv_bfloat16>(void* dst, size_t i, float v) {
    static_cast<__nv_bfloat16*>(dst)[i] = __float2bfloat16_rn(v);
}

// One 16-byte chunk of activation-type values <-> float32.
template <typename T> struct Chunk;
template <> struct Chunk<float> {
    static constexpr int kN = 4;
    static __device__ __forceinline__ void unpack(const uint4& c, float* v) {
        v[0] = __uint_as_float(c.x); v[1] = __uint_as_float(c.y); v[2] = __uint_as_float(c.z); v[3] = __uint_as_float(c.w);
    }
    static __device__ __forceinline__ uint4 pack(const float* v) {
        return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
    }
};
template <> struct Chunk<__nv_bfloat16> {
    static constexpr int kN = 8;
    static __device__ __forceinline__ void unpack(const uint4& c, float* v) {
        const unsigned w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) { v[2 * q] = __uint_as_float(w[q] << 16); v[2 * q + 1] = __uint_as_float(w[q] & 0xffff0000u); }
    }
    static __device__ __forceinline__ uint4 pack(const float* v) {
        unsigned w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const unsigned lo = __bfloat16_as_ushort(__float2bfloat16_rn(v[2 * q]));
            const unsigned hi = __bfloat16_as_ushort(__float2bfloat16_rn(v[2 * q + 1]));
            w[q] = lo | (hi << 16);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// The activation rows of this pass, transformed on the way into shared memory (ActOp).  Called by
// every thread of the CTA; all of them share each row (with one row per pass, one warp per row
// would leave the rest of the CTA waiting for it).
template <typename T, int MROWS>
__device__ void load_rows_transformed(const GemvParams& p, uint4* xs, int x_stride, int nch) {
    constexpr int N = Chunk<T>::kN;
    constexpr int kNW = kThreads / 32;
    __shared__ float s_ss[MROWS][kNW];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const ActOp& a = p.act;
    int src[MROWS];                                     // source row of x, -1: the row is all zero
#pragma unroll
    for (int m = 0; m < MROWS; ++m) {
        const int row = p.m0 + m;
        int sr = -1;
        if (m < p.mcount) {
            sr = row;
            if (p.x_rows != nullptr) {
                sr = p.x_rows[row];
                if (sr < 0 || sr >= p.x_row_count) {
                    if (tid == 0) report_error(p.status, CTCSD_ERR_INVALID_ARG, row);
                    sr = -1;
                }
            }
            if (a.op == 1 && a.n_new != nullptr && sr >= 0) {
                int r = a.n_new[sr / a.R];
                r = r < 0 ? 0 : (r > a.R ? a.R : r);
                if (sr - (sr / a.R) * a.R >= r) sr = -1;                 // not a live row
            }
        }
        src[m] = sr;
    }
    float v[N];
    if (a.op == 3) {
        for (int i = tid; i < MROWS * nch; i += kThreads) {
            const int m = i / nch, ch = i - m * nch;
            uint4 out = make_uint4(0, 0, 0, 0);
            if (m < p.mcount) {
                const float* g = a.gu + (size_t)(p.m0 + m) * 2 * p.H + (size_t)ch * N;
                const float* u = g + p.H;
#pragma unroll
                for (int q = 0; q < N; ++q) v[q] = g[q] / (1.f + __expf(-g[q])) * u[q];
                out = Chunk<T>::pack(v);
            }
            xs[(size_t)m * x_stride + ch] = out;
        }
        return;
    }
    float ss[MROWS];
#pragma unroll
    for (int m = 0; m < MROWS; ++m) {
        ss[m] = 0.f;
        if (src[m] < 0) continue;
        const int row = p.m0 + m;
        const uint4* xrow = reinterpret_cast<const uint4*>(p.x) + (size_t)src[m] * nch;
        const float* add = (a.op == 2) ? a.add + (size_t)row * p.H : nullptr;
        float* sum_out = (a.op == 2 && a.sum_out != nullptr && blockIdx.x == 0) ? a.sum_out + (size_t)row * p.H : nullptr;
        for (int ch = tid; ch < nch; ch += kThreads) {
            Chunk<T>::unpack(xrow[ch], v);
#pragma unroll
            for (int q = 0; q < N; ++q) {
                if (add) v[q] += add[ch * N + q];
                if (sum_out) sum_out[ch * N + q] = v[q];
                ss[m] += v[q] * v[q];
            }
        }
    }
#pragma unroll
    for (int m = 0; m < MROWS; ++m) {
        const float w = warp_sum(ss[m]);
        if (lane == 0) s_ss[m][warp] = w;
    }
    __syncthreads();
#pragma unroll
    for (int m = 0; m < MROWS; ++m) {
        uint4* dst = xs + (size_t)m * x_stride;
        if (src[m] < 0) {
            for (int ch = tid; ch < nch; ch += kThreads) dst[ch] = make_uint4(0, 0, 0, 0);
            continue;
        }
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < kNW; ++w) tot += s_ss[m][w];
        const float inv = rsqrtf(tot / (float)p.H + a.eps);
        const int row = p.m0 + m;
        const uint4* xrow = reinterpret_cast<const uint4*>(p.x) + (size_t)src[m] * nch;
        const float* add = (a.op == 2) ? a.add + (size_t)row * p.H : nullptr;
        for (int ch = tid; ch < nch; ch += kThreads) {
            Chunk<T>::unpack(xrow[ch], v);
#pragma unroll
            for (int q = 0; q < N; ++q) {
                if (add) v[q] += add[ch * N + q];
                v[q] = v[q] * inv * a.gain[ch * N + q];
            }
            dst[ch] = Chunk<T>::pack(v);
        }
    }
}

// One CTA per SM.  Warp 8 is the producer: it walks the CTA's contiguous range of weight rows
// and copies G rows (about 64 KB: the copy engine's cost per copy is high) per ring slot with
// the bulk-copy engine, as far ahead as the ring allows.  Warps 0..7 consume the slots in
// order.
//   bfloat16: the warps split the hidden axis.  Each warp multiplies its share of all G rows
//   with the activation rows on the tensor cores (mma.m16n8k16: the 16 "M" rows are weight
//   rows, the 8 "N" columns are activation rows, so up to 8 activation rows cost the same as
//   one); the per-warp partial sums go to a small ring in shared memory, from which warps
//   9..12 (the epilogue) add them up and fold the logits into the running states, off the
//   consumers' critical path.
//   float32: each warp owns whole rows of the slot, uses fused multiply-adds and folds its own
//   logits.
// The running (max, sum of exp, best-8) states are held by the threads that own a (weight row
// of the slot, activation row) pair; they are merged per CTA at the end and per grid by the CTA
// that finishes last.
template <typename T, int MROWS>
__global__ void __launch_bounds__(kThreads, 1) gemv_stream_kernel(GemvParams p, int nslots, int G) {
    constexpr bool kMma = sizeof(T) == 2;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const int row_bytes = p.H * (int)sizeof(T);
    const int nch = row_bytes / 16;                                  // 16-byte chunks per row
    const int slot_bytes = G * row_bytes;
    // activation rows are padded by 64 bytes so that neighbouring rows start in different banks
    const int x_stride = nch + 4;                                    // in 16-byte chunks
    uint4* xs = reinterpret_cast<uint4*>(smem_raw);                  // [MROWS][x_stride]
    unsigned char* ring = smem_raw + (size_t)MROWS * x_stride * 16;  // [nslots][G][row_bytes]
    RingShared* sh = reinterpret_cast<RingShared*>(ring + (size_t)nslots * slot_bytes);
    __shared__ DraftPartial s_part[2][kStateRows][MROWS];
    // per-warp partial sums of a fill (bf16 path).  With eight activation rows their copies in shared
    // memory leave the weight ring the less room: two buffers instead of four buy an eighth row per slot.
    constexpr int kCD = MROWS == 8 ? 2 : kCDepth;
    __shared__ float s_cpart[kCD][kWarps][16][8];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int* abort_flag = &sh->abort_flag;

    if (tid == 0) {
        for (int s = 0; s < nslots; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], kWarps); }
        for (int d = 0; d < kCD; ++d) { tc::mbar_init(&sh->cfull[d], kWarps); tc::mbar_init(&sh->cempty[d], kEpiWarps); }
        sh->abort_flag = 0;
        sh->never_set = 0;
        sh->is_last = 0;
        tc::fence_barrier_init();
    }
    __syncthreads();                                                 // the barriers exist

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

    // producer state (used by lane 0 of warp 8 only)
    const uint64_t policy = tc::policy_evict_first();
    bool prod_ok = true;
    int prod_j = 0;
    auto issue_fill = [&](int j) -> bool {
        const int s = j % nslots;
        const uint32_t ph = (uint32_t)(j / nslots) & 1u;
        if (!tc::mbar_wait(&sh->empty[s], ph ^ 1u, abort_flag)) return false;
        const int rows = (ntotal - j * G < G) ? ntotal - j * G : G;
        const uint32_t bytes = (uint32_t)rows * (uint32_t)row_bytes;
        // never hand the copy engine a range outside the weights or the ring
        const long long first = r0 + (long long)j * G;
        if (rows < 1 || first < 0 || first + rows > R || (bytes & 15u) != 0 || bytes > (uint32_t)slot_bytes) {
            report_error(p.status, CTCSD_ERR_INTERNAL, 12);
            return false;
        }
        tc::mbar_arrive_expect_tx(&sh->full[s], bytes);
        tc::bulk_load_1d(ring + (size_t)s * slot_bytes, Wbase + (size_t)first * row_bytes, bytes, &sh->full[s], policy);
        return true;
    };
    // The weights are never written by any kernel, so the ring is filled before this kernel waits
    // for its predecessor in the stream: the copies run while the predecessor drains.
    if (warp == kWarps && lane == 0) {
        for (; prod_j < nfill && prod_j < nslots && prod_ok; ++prod_j) prod_ok = issue_fill(prod_j);
        if (!prod_ok) --prod_j;
    }
    // everything above touches only the weights and this CTA's shared memory; the activations
    // below may come from the kernel that precedes this one in the stream
    pdl_wait();
    pdl_trigger();
    if (p.act.op != 0) load_rows_transformed<T, MROWS>(p, xs, x_stride, nch);
    else for (int i = tid; i < MROWS * nch; i += kThreads) {
        int m = i / nch, ch = i - m * nch;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (m < p.mcount) {
            int src = p.m0 + m;
            if (p.x_rows != nullptr) {
                src = p.x_rows[p.m0 + m];
                if (src < 0 || src >= p.x_row_count) {               // a row map that leaves x: read nothing
                    if (ch == 0) report_error(p.status, CTCSD_ERR_INVALID_ARG, p.m0 + m);
                    src = -1;
                }
            }
            if (src >= 0) v = reinterpret_cast<const uint4*>(p.x)[(size_t)src * nch + ch];
        }
        xs[m * x_stride + ch] = v;
    }
    for (int i = tid; i < 2 * kStateRows * MROWS; i += kThreads) {   // states nobody fills stay empty
        DraftPartial* d = &s_part[0][0][0] + i;
        d->mx = -INFINITY;
        d->sum = 0.f;
#pragma unroll
        for (int q = 0; q < kTopSlots; ++q) { d->val[q] = -INFINITY; d->id[q] = INT_MAX; }
    }
    __syncthreads();

    if (warp == kWarps) {
        // ---------------- producer ----------------
        if (lane == 0) {
            bool ok = prod_ok;
            int j = prod_j;
            for (; j < nfill && ok; ++j) {
                ok = issue_fill(j);
                if (!ok) break;
            }
            if (!ok) {
                if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 10);
                *abort_flag = 1;
            }
            // All of this CTA's weights are requested.  If the caller named a range that the next
            // heavy kernel will stream, ask L2 for this CTA's share of it now: the fetch runs
            // while the small kernels that follow leave HBM idle.
            if (ok && p.pf_bytes != 0) {
                const unsigned long long chunk = 64 * 1024;
                const unsigned long long nchunks = (p.pf_bytes + chunk - 1) / chunk;
                for (unsigned long long c = blockIdx.x; c < nchunks; c += gridDim.x) {
                    unsigned long long len = p.pf_bytes - c * chunk;
                    if (len > chunk) len = chunk;
                    len &= ~15ull;
                    if (len) tc::bulk_prefetch_l2(static_cast<const unsigned char*>(p.pf_ptr) + c * chunk, (uint32_t)len);
                }
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
        // ---------------- consumers (warps 0..7) and epilogue (warps 9..12) ----------------
        // Every warp visits every fill in order and arrives on the barriers it takes part in, so
        // no warp is ever more than one phase away from a barrier it waits on (a parity wait
        // means nothing to a waiter that is further behind).
        const bool is_epi = warp > kWarps;
        if (kMma ? true : !is_epi) {
            RunState st;
            st.init();
            int cur_seg = 0;
            // the (row of the slot, activation row) pair whose state this thread keeps
            const int epi_idx = (warp - kWarps - 1) * 32 + lane;
            const int own_r = kMma ? (epi_idx >> 3) : warp;
            const int own_m = kMma ? (epi_idx & 7) : lane;
            const bool owner = kMma ? (is_epi && own_m < p.mcount) : (lane < p.mcount);
            float bias = 0.f;
            if (owner && p.blank_bias != nullptr) {
                const int row = p.m0 + own_m;
                bias = p.blank_bias[p.row_seq ? p.row_seq[row] : row];
            }
            // sampling acceptance (LM head only): this thread's activation row is a tree node, whose
            // depth picks the noise row
            const float* noise_row = nullptr;
            if (owner && p.sn.noise != nullptr) {
                const int row = p.m0 + own_m;
                int d = p.sn.depth[row];
                d = d < 0 ? 0 : (d >= p.sn.rows_per_seq ? p.sn.rows_per_seq - 1 : d);
                noise_row = p.sn.noise + ((size_t)(row / p.sn.max_nodes) * p.sn.rows_per_seq + d) * (size_t)rps;
            }
            auto push_logit = [&](float z, int i) {          // i: row of the CTA's range
                const int seg = i >= n_seg0 ? 1 : 0;
                if (seg != cur_seg) {                         // this thread's rows now belong to the next slot
                    st.store(&s_part[0][own_r][own_m]);
                    st.init();
                    cur_seg = 1;
                }
                const int slot = slot0 + seg;
                const int v = (int)(r0 + i - (long long)slot * rps);
                if (v == (int)rps - 1) z += bias;
                const size_t at = ((size_t)(p.m0 + own_m) * p.slots + slot) * rps + v;
                if (p.mode == 2) {                             // plain product (plus, if asked, a residual): it is the output
                    if (p.plain_add) z += p.plain_add[at];
                    if (p.logits_dbg) p.logits_dbg[at] = z;
                    if (p.plain_out_t) store_as<T>(p.plain_out_t, at, z);
                    return;
                }
                if (p.logits_dbg) p.logits_dbg[at] = z;
                if (noise_row != nullptr) z = __fmaf_rn(z, p.sn.inv_temp, noise_row[v]);
                st.push(z, v);
            };

            bool failed = false;
            for (int j = 0; j < nfill; ++j) {
                const int rows = (ntotal - j * G < G) ? ntotal - j * G : G;
                const int d = j % kCD;
                const uint32_t dph = (uint32_t)(j / kCD) & 1u;
                if (kMma && is_epi) {
                    // ---- epilogue: add the eight partial sums, fold the logit into the state ----
                    if (!tc::mbar_wait(&sh->cfull[d], dph, abort_flag)) { failed = true; break; }
                    if (owner && own_r < rows) {
                        float z = 0.f;
#pragma unroll
                        for (int w = 0; w < kWarps; ++w) z += s_cpart[d][w][own_r][own_m];
                        push_logit(z, j * G + own_r);
                    }
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(&sh->cempty[d]);
                    continue;
                }
                const int s = j % nslots;
                const uint32_t ph = (uint32_t)(j / nslots) & 1u;
                if (!tc::mbar_wait(&sh->full[s], ph, abort_flag)) { failed = true; break; }
                const unsigned char* slot_base = ring + (size_t)s * slot_bytes;
                if constexpr (kMma) {
                    const int g = lane >> 2, t = lane & 3;
                    const uint4* rowA = reinterpret_cast<const uint4*>(slot_base + (size_t)g * row_bytes);
                    const uint4* rowB = reinterpret_cast<const uint4*>(slot_base + (size_t)(g + 8) * row_bytes);
                    const bool hasA = g < rows, hasB = g + 8 < rows, hasX = g < MROWS;
                    const uint4* xrow = xs + (hasX ? g : 0) * x_stride;
                    // A block of 32 hidden elements = four 16-byte chunks, one per thread of a quad;
                    // the k index inside a block is permuted the same way for weights and activations.
                    // Four blocks are in flight at a time, each with its own accumulators, so that
                    // neither the loads nor the dependent tensor-core instructions serialise.
                    constexpr int kU = 4;
                    float cc[kU][4], ce[kU][4];                 // (the two halves of a block accumulate apart: shorter chains)
#pragma unroll
                    for (int u = 0; u < kU; ++u) {
                        cc[u][0] = cc[u][1] = cc[u][2] = cc[u][3] = 0.f;
                        ce[u][0] = ce[u][1] = ce[u][2] = ce[u][3] = 0.f;
                    }
                    for (int kb0 = warp; kb0 * 4 < nch; kb0 += kWarps * kU) {      // the same trip count for all lanes
                        uint4 P[kU], Q[kU], X[kU];
#pragma unroll
                        for (int u = 0; u < kU; ++u) {
                            const int ch = (kb0 + u * kWarps) * 4 + t;
                            const bool in = ch < nch;
                            const uint4 z4 = make_uint4(0, 0, 0, 0);
                            P[u] = (hasA && in) ? rowA[ch] : z4;
                            Q[u] = (hasB && in) ? rowB[ch] : z4;
                            X[u] = (hasX && in) ? xrow[ch] : z4;
                        }
#pragma unroll
                        for (int u = 0; u < kU; ++u) {
                            mma_16816(cc[u], P[u].x, Q[u].x, P[u].y, Q[u].y, X[u].x, X[u].y);
                            mma_16816(ce[u], P[u].z, Q[u].z, P[u].w, Q[u].w, X[u].z, X[u].w);
                        }
                    }
                    // the accumulators depend on every load of the slot: it can be refilled
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(&sh->empty[s]);
                    // c0,c1: weight row g x activation rows 2t,2t+1;  c2,c3: weight row g+8
                    if (!tc::mbar_wait(&sh->cempty[d], dph ^ 1u, abort_flag)) { failed = true; break; }
#pragma unroll
                    for (int u = 0; u < kU; ++u) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) cc[u][q] += ce[u][q];
                    }
                    float* cp = &s_cpart[d][warp][0][0];
                    *reinterpret_cast<float2*>(cp + g * 8 + 2 * t) =
                        make_float2((cc[0][0] + cc[1][0]) + (cc[2][0] + cc[3][0]), (cc[0][1] + cc[1][1]) + (cc[2][1] + cc[3][1]));
                    *reinterpret_cast<float2*>(cp + (g + 8) * 8 + 2 * t) =
                        make_float2((cc[0][2] + cc[1][2]) + (cc[2][2] + cc[3][2]), (cc[0][3] + cc[1][3]) + (cc[2][3] + cc[3][3]));
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(&sh->cfull[d]);
                } else {
                    float zrow[kRowsPerWarp];
                    int nmine = 0;
#pragma unroll
                    for (int q = 0; q < kRowsPerWarp; ++q) {
                        const int rin = warp + q * kWarps;          // row within the slot
                        zrow[q] = 0.f;
                        if (rin < rows) {
                            const uint4* wrow = reinterpret_cast<const uint4*>(slot_base + (size_t)rin * row_bytes);
                            float acc[MROWS];
#pragma unroll
                            for (int m = 0; m < MROWS; ++m) acc[m] = 0.f;
#pragma unroll 4
                            for (int ch = lane; ch < nch; ch += 32) {
                                const uint4 w = wrow[ch];
#pragma unroll
                                for (int m = 0; m < MROWS; ++m) acc[m] = Elem<T>::dot(w, xs[m * x_stride + ch], acc[m]);
                            }
#pragma unroll
                            for (int m = 0; m < MROWS; ++m) {
                                const float v = warp_sum(acc[m]);
                                if (lane == m) zrow[q] = v;
                            }
                            nmine = q + 1;
                        }
                    }
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(&sh->empty[s]);
#pragma unroll
                    for (int q = 0; q < kRowsPerWarp; ++q)
                        if (q < nmine && owner) push_logit(zrow[q], j * G + warp + q * kWarps);
                }
            }
            if (failed && lane == 0) {
                if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 11);
                *abort_flag = 1;
            }
            if (owner) {
                if (cur_seg == 0) {
                    st.store(&s_part[0][own_r][own_m]);
                    st.init();
                }
                st.store(&s_part[1][own_r][own_m]);
            }
        }
    }
    __syncthreads();
    if (p.mode == 2) return;                                         // no selection, nothing to merge

    // fold the CTA's states per segment: warp m merges activation row m's states, one per lane
    for (int seg = 0; seg < 2; ++seg) {
        if (warp < MROWS) {
            RunState ms;
            ms.init();
            if (lane < kStateRows) ms.absorb(s_part[seg][lane][warp]);
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
        // The CTAs whose row range touches this slot are a contiguous interval that follows from
        // the partition formula, so a lane goes straight to "its" CTA's state: one memory latency
        // instead of a scan over all CTAs' slot tags (the tag is still checked: a CTA marks a
        // segment without rows as unused).
        const long long g = gridDim.x;
        const long long lo_row = (long long)slot * rps, hi_row = lo_row + rps;     // the slot's rows
        long long c_lo = lo_row * g / R, c_hi = hi_row * g / R;
        while (c_lo > 0 && R * c_lo / g > lo_row) --c_lo;                          // first CTA with r1 > lo_row
        while (c_lo < g - 1 && R * (c_lo + 1) / g <= lo_row) ++c_lo;
        if (c_hi > g - 1) c_hi = g - 1;
        while (c_hi > 0 && R * c_hi / g >= hi_row) --c_hi;                         // last CTA with r0 < hi_row
        for (long long c = c_lo + lane; c <= c_hi; c += 32) {
            const int seg = slot - (int)((R * c / g) / rps);
            if (seg < 0 || seg > 1) continue;
            const int e = (int)(2 * c + seg);
            const int tag = __ldcg(p.part_slot + e);
            DraftPartial q = load_partial_cg(p.part + (size_t)m * p.grid * 2 + e);
            if (tag == slot) fs.absorb(q);
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
    // dynamic shared memory per CTA: what the device allows minus the kernel's static part
    cudaFuncAttributes fa;
    CTCSD_CUDA_CHECK(h, cudaFuncGetAttributes(&fa, kern));
    int optin = 0;
    CTCSD_CUDA_CHECK(h, cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, h->device));
    if ((size_t)optin < fa.sharedSizeBytes + 32 * 1024) return CTCSD_ERR_UNSUPPORTED;
    size_t budget = (size_t)optin - fa.sharedSizeBytes - 2048;
    if (budget > 208 * 1024) budget = 208 * 1024;
    const size_t fixed = (size_t)MROWS * (row_bytes + 64) + sizeof(RingShared);
    // rows per ring slot: copies of 64 KB and more keep the copy engine busiest (its cost per copy is
    // large), as long as at least two slots fit.  bfloat16: the consumers are bound by the rate at
    // which the tensor-core instructions issue, and a slot costs the same number of them for 1 to
    // 16 rows, so slots of 80 KB (two of them) beat three of 64 KB: 10 / 9 / 8 rows of 8 KB per slot
    // gave 193 / 197 / 200 us for the 7B draft head and 282 / 286 / 297 us for the step; 12 rows no more.
    int G = (int)(((sizeof(T) == 2 ? 80 : 64) * 1024) / row_bytes);
    if (G < 1) G = 1;
    if (G > kWarps * kRowsPerWarp) G = kWarps * kRowsPerWarp;
    // bfloat16: a tensor-core step costs the same for 1 to 16 weight rows, and a slot's steps are a
    // chain whose length grows with the row: long rows get at least four rows per slot
    if (sizeof(T) == 2 && G < 4) G = 4;
    while (G > 1 && fixed + 2 * (size_t)G * row_bytes > budget) --G;
    const size_t slot_bytes = (size_t)G * row_bytes;
    if (fixed + slot_bytes > budget) return CTCSD_ERR_UNSUPPORTED;
    long long nslots = (long long)((budget - fixed) / slot_bytes);
    if (nslots > kMaxSlots) nslots = kMaxSlots;
    const size_t smem = fixed + (size_t)nslots * slot_bytes;
    CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    long long R = (long long)p.slots * p.rows_per_slot;
    long long grid = h->num_sms;
    if (grid > R) grid = R;
    if (grid < p.slots) grid = p.slots;         // a CTA's range then touches at most two slots
    p.grid = (int)grid;
    CTCSD_CUDA_CHECK(h, launch_pdl(kern, dim3((unsigned)grid), dim3(kThreads), smem, stream, 1, p, (int)nslots, G));
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}

// bfloat16 rows go through the tensor-core consumer, up to 8 activation rows per pass over the
// weights; float32 rows through the fused-multiply-add consumer, up to 4 per pass.
int launch_typed_bf16(Handle* h, cudaStream_t stream, int M, GemvParams& p) {
    // the activation rows of a pass sit in shared memory beside the weight ring: with a long inner
    // dimension fewer rows go into a pass, so that the ring keeps at least two slots of useful size
    int per_pass = 8;
    while (per_pass > 1 && (size_t)per_pass * p.H * 2 > 96 * 1024) per_pass >>= 1;
    for (int m0 = 0; m0 < M; m0 += per_pass) {
        p.m0 = m0;
        p.mcount = (M - m0 < per_pass) ? (M - m0) : per_pass;
        int rc;
        if (p.mcount == 1) rc = launch_one<__nv_bfloat16, 1>(h, stream, p);
        else if (p.mcount == 2) rc = launch_one<__nv_bfloat16, 2>(h, stream, p);
        else if (p.mcount <= 4) rc = launch_one<__nv_bfloat16, 4>(h, stream, p);
        else rc = launch_one<__nv_bfloat16, 8>(h, stream, p);
        if (rc != CTCSD_OK) return rc;
    }
    return CTCSD_OK;
}

int launch_typed_f32(Handle* h, cudaStream_t stream, int M, GemvParams& p) {
    int per_pass = 4;
    while (per_pass > 1 && (size_t)per_pass * p.H * 4 > 96 * 1024) per_pass >>= 1;
    for (int m0 = 0; m0 < M; m0 += per_pass) {
        p.m0 = m0;
        p.mcount = (M - m0 < per_pass) ? (M - m0) : per_pass;
        int rc;
        if (p.mcount == 1) rc = launch_one<float, 1>(h, stream, p);
        else if (p.mcount == 2) rc = launch_one<float, 2>(h, stream, p);
        else rc = launch_one<float, 4>(h, stream, p);
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
    if (p.mode != 0) { p.pf_ptr = nullptr; p.pf_bytes = 0; }
    if (dtype == CTCSD_DTYPE_BF16) return launch_typed_bf16(h, stream, M, p);
    return launch_typed_f32(h, stream, M, p);
}

}  // namespace ctcsd
