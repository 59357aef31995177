// Shared host/device declarations for the ctcsd kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "ctcsd.h"

namespace ctcsd {

// ---------------------------------------------------------------------------------------
// Workspace layout.  Everything the kernels need beyond their inputs and outputs lives in
// the caller's workspace at the offsets computed here.
// ---------------------------------------------------------------------------------------
constexpr int kTopSlots = CTCSD_MAX_K;          // every partial top-k list keeps 8 entries

// Partial result of one chunk of vocabulary rows for one (row m, slot t):
// running max, sum of exp(z - max), and the chunk's best kTopSlots logits with their ids.
struct alignas(16) DraftPartial {
    float mx;
    float sum;
    float val[kTopSlots];
    int   id[kTopSlots];
    int   pad[2];
};
static_assert(sizeof(DraftPartial) == 80, "DraftPartial is copied as five 16-byte words");

struct Layout {
    size_t status_off;        // int[16]: [0] status word, [1] detail
    size_t counter_off;       // unsigned[kCounters]: "chunks finished" tickets, zero between calls
    size_t zeroed_bytes;      // everything below this offset is cleared when the handle is created
    size_t draft_part_off;    // DraftPartial[8][gemv_grid_max][2]  (weight-streaming GEMV partials)
    size_t part_slot_off;     // int[gemv_grid_max][2]
    size_t lm_key_off;        // uint64[lm_key_count]: packed (logit, id) row maxima of the tensor-core LM head, zero between calls
    size_t seq_ticket_off;    // unsigned[B]: per-sequence "CTAs finished" tickets of the history update, zero between calls
    size_t tc_part_off;       // DraftPartial[T * tiles_per_slot][rows padded to 128]: tensor-core draft head (only if max_draft_rows > 8)
    size_t tc_part_bytes;
    size_t lm_rows_off;       // act[lm_key_count][H]: the LM head's live activation rows packed densely (bf16, more than 128 tree rows)
    size_t lm_rowmap_off;     // int[lm_key_count + 1]: packed row -> tree row; the last entry is the number of live rows
    size_t total;
    int gemv_grid_max;        // largest grid the GEMV may use
    int lm_key_count;
};

constexpr int kCounters = 64;

struct Handle {
    ctcsd_config cfg;
    Layout lay;
    char* ws;
    int device;
    int num_sms;
    int last_cuda_error;
    long long launches;
    const void* l2_hint_ptr;     // range that ctcsd_draft_logits asks L2 to fetch when it finishes
    size_t l2_hint_bytes;
};

// Sampling acceptance: the token drawn after tree node i of sequence b is
// argmax_v fma(y[v], inv_temp, noise[(b * rows_per_seq + depth[b,i]) * V + v]).  noise == null: plain arg-max.
struct SampleNoise {
    const float* noise;      // [B][rows_per_seq][V] standard Gumbel noise, or null
    const int* depth;        // [B*max_nodes] tree depth of every node
    int max_nodes;
    int rows_per_seq;        // T + 1
    float inv_temp;
};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

Layout make_layout(const ctcsd_config& cfg, int num_sms);
int validate_config(const ctcsd_config& cfg);

#define CTCSD_CUDA_CHECK(h, expr)                                   \
    do {                                                            \
        cudaError_t e__ = (expr);                                   \
        if (e__ != cudaSuccess) {                                   \
            (h)->last_cuda_error = (int)e__;                        \
            return CTCSD_ERR_CUDA;                                  \
        }                                                           \
    } while (0)

#define CTCSD_LAUNCH_CHECK(h)                                       \
    do {                                                            \
        (h)->launches++;                                            \
        CTCSD_CUDA_CHECK(h, cudaGetLastError());                    \
    } while (0)

#ifdef __CUDACC__
// Launches `kernel` with the programmatic-dependent-launch attribute (and, if cluster_x > 1, as
// thread-block clusters of that many CTAs along x).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                              int cluster_x, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int na = 0;
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
    if (cluster_x > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)cluster_x;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = (unsigned)na;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

inline int* status_ptr(const Handle* h) { return reinterpret_cast<int*>(h->ws + h->lay.status_off); }
inline unsigned* counter_ptr(const Handle* h) { return reinterpret_cast<unsigned*>(h->ws + h->lay.counter_off); }

// ---------------------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// L2 policy "evict first": a stream that is read once must not push the step's small,
// reused data (K/V cache, activations, code) out of L2.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// 16-byte streaming load: no L1 allocation, L2 eviction priority given by `policy`.
__device__ __forceinline__ uint4 ld_stream16(const void* p, uint64_t policy) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0,%1,%2,%3}, [%4], %5;"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p), "l"(policy));
    return r;
}

// A 32-bit word holding two bfloat16 -> two floats (low half first).
__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// "a ranks before b" for (logit, id) pairs: larger logit first, equal logits -> lower id.
__device__ __forceinline__ bool ranks_before(float va, int ia, float vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}

// Insert (v, id) into a descending list of kTopSlots entries held in registers.
__device__ __forceinline__ void topk_insert(float (&val)[kTopSlots], int (&id)[kTopSlots], float v, int i) {
    if (!ranks_before(v, i, val[kTopSlots - 1], id[kTopSlots - 1])) return;
#pragma unroll
    for (int s = kTopSlots - 1; s >= 0; --s) {
        bool shift = (s > 0) && ranks_before(v, i, val[s - 1], id[s - 1]);
        bool here = !shift && ranks_before(v, i, val[s], id[s]);
        float pv = (s > 0) ? val[s - 1] : 0.f;
        int pi = (s > 0) ? id[s - 1] : 0;
        if (shift) { val[s] = pv; id[s] = pi; }
        else if (here) { val[s] = v; id[s] = i; }
    }
}

// The same with only the first KS entries of the list in use (the others stay at their initial
// "nothing" value): a caller that needs at most KS winners pays for KS slots.
template <int KS>
__device__ __forceinline__ void topk_insert_n(float (&val)[kTopSlots], int (&id)[kTopSlots], float v, int i) {
    static_assert(KS >= 1 && KS <= kTopSlots, "slot count");
    if (!ranks_before(v, i, val[KS - 1], id[KS - 1])) return;
#pragma unroll
    for (int s = KS - 1; s >= 0; --s) {
        bool shift = (s > 0) && ranks_before(v, i, val[s - 1], id[s - 1]);
        bool here = !shift && ranks_before(v, i, val[s], id[s]);
        float pv = (s > 0) ? val[s - 1] : 0.f;
        int pi = (s > 0) ? id[s - 1] : 0;
        if (shift) { val[s] = pv; id[s] = pi; }
        else if (here) { val[s] = v; id[s] = i; }
    }
}

// Programmatic dependent launch.  Every kernel of the step is launched so that it may start
// while its predecessor in the stream is still draining: what it does before pdl_wait() (set
// up shared memory and barriers, prefetch weights, which no kernel ever writes) overlaps with the
// predecessor's tail.  pdl_wait() returns once the predecessor grid has completed and its
// writes are visible; nothing that a predecessor produces may be read, and no global memory
// may be written, before it.  Every kernel calls it, which orders the whole chain.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Lets the next kernel in the stream begin to launch (it still waits in its own pdl_wait()).
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ void report_error(int* status, int code, int detail) {
    if (atomicCAS(status, 0, code) == 0) status[1] = detail;
}

// Debug build (-DCTCSD_DEBUG_BOUNDS): an index check at the places where a kernel forms the index
// of a store into a caller's array or into a list in shared memory.  A check that fails records
// CTCSD_ERR_INTERNAL and 1000 + the site number in the device status word and the store is
// skipped; nothing traps.  In the normal build the checks compile to nothing (the production
// guards - clamped counts, `row < M` tests and the like - are always there).
#ifdef CTCSD_DEBUG_BOUNDS
__device__ __forceinline__ bool debug_in_bounds(int* status, int site, long long idx, long long n) {
    if (idx >= 0 && idx < n) return true;
    if (status != nullptr) report_error(status, CTCSD_ERR_INTERNAL, 1000 + site);
    return false;
}
#define CTCSD_IN_BOUNDS(status, site, idx, n) ctcsd::debug_in_bounds((status), (site), (long long)(idx), (long long)(n))
#else
#define CTCSD_IN_BOUNDS(status, site, idx, n) true
#endif

#endif  // __CUDACC__

}  // namespace ctcsd

// The opaque handle of the C ABI wraps the C++ state.
struct ctcsd_handle {
    ctcsd::Handle h;
};
