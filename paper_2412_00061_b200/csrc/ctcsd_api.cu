// Handle management, configuration checks and workspace layout for the ctcsd C ABI.
#include "common.cuh"
#include "lm_head_tc.cuh"

#include <stdlib.h>
#include <string.h>
#include <new>

namespace ctcsd {

int validate_config(const ctcsd_config& c) {
    if (c.B < 1 || c.H < 8 || c.H % 8 != 0 || c.V < 1) return CTCSD_ERR_INVALID_ARG;
    if (c.T < 1 || c.T > CTCSD_MAX_T || c.k < 1 || c.k > CTCSD_MAX_K) return CTCSD_ERR_INVALID_ARG;
    if (c.k > c.V + 1 || c.T * c.k > 64) return CTCSD_ERR_INVALID_ARG;
    if (c.beam < 0 || c.beam > CTCSD_MAX_BEAM) return CTCSD_ERR_INVALID_ARG;
    if (c.beam == 0) {
        long long paths = 1;
        for (int t = 0; t < c.T; ++t) paths *= c.k;
        if (paths > CTCSD_MAX_PATHS) return CTCSD_ERR_INVALID_ARG;
    }
    if (c.topN < 1 || c.topN > CTCSD_MAX_TOPN) return CTCSD_ERR_INVALID_ARG;
    if (c.max_nodes < 2 || c.max_nodes > CTCSD_MAX_NODES) return CTCSD_ERR_INVALID_ARG;
    if (c.Hq < 1 || c.Hkv < 1 || c.Hq % c.Hkv != 0) return CTCSD_ERR_INVALID_ARG;
    if (c.D != 64 && c.D != 128) return CTCSD_ERR_INVALID_ARG;
    if (c.dtype != CTCSD_DTYPE_F32 && c.dtype != CTCSD_DTYPE_BF16) return CTCSD_ERR_INVALID_ARG;
    if (c.score_mode != CTCSD_SCORE_SUM && c.score_mode != CTCSD_SCORE_MAX) return CTCSD_ERR_INVALID_ARG;
    if (c.score_mode == CTCSD_SCORE_MAX && c.beam != 0) return CTCSD_ERR_UNSUPPORTED;
    if (c.max_draft_rows < 0) return CTCSD_ERR_INVALID_ARG;
    if ((long long)c.B * c.max_nodes > (1 << 20)) return CTCSD_ERR_INVALID_ARG;
    return CTCSD_OK;
}

Layout make_layout(const ctcsd_config& c, int num_sms) {
    Layout l;
    memset(&l, 0, sizeof(l));
    size_t off = 0;
    l.status_off = off;      off = align_up(off + 16 * sizeof(int), 256);
    l.counter_off = off;     off = align_up(off + kCounters * sizeof(unsigned), 256);
    l.lm_key_count = (c.B * c.max_nodes + 127) / 128 * 128;
    l.lm_key_off = off;      off = align_up(off + sizeof(unsigned long long) * (size_t)l.lm_key_count, 256);
    l.seq_ticket_off = off;  off = align_up(off + sizeof(unsigned) * (size_t)c.B, 256);
    l.zeroed_bytes = off;
    l.gemv_grid_max = num_sms * 8 > 64 ? num_sms * 8 : 64;
    l.draft_part_off = off;  off = align_up(off + sizeof(DraftPartial) * 8 * (size_t)l.gemv_grid_max * 2, 256);
    l.part_slot_off = off;   off = align_up(off + sizeof(int) * (size_t)l.gemv_grid_max * 2, 256);
    {
        const int rows = c.max_draft_rows > 0 ? c.max_draft_rows : c.B;
        l.tc_part_off = off;
        l.tc_part_bytes = 0;
        if (rows > 8 && c.dtype == CTCSD_DTYPE_BF16) {
            const int classes = c.V + 1;
            const int nt = classes >= 224 ? 224 : (classes + 15) / 16 * 16;
            const size_t tiles = (size_t)c.T * ((classes + nt - 1) / nt);
            l.tc_part_bytes = sizeof(DraftPartial) * tiles * kDraftColSplit * (size_t)((rows + 127) / 128 * 128);
            off = align_up(off + l.tc_part_bytes, 256);
        }
    }
    l.lm_rows_off = l.lm_rowmap_off = off;
    if (c.dtype == CTCSD_DTYPE_BF16 && c.B * c.max_nodes > 128) {
        l.lm_rows_off = off;    off = align_up(off + (size_t)l.lm_key_count * c.H * 2, 256);
        l.lm_rowmap_off = off;  off = align_up(off + sizeof(int) * ((size_t)l.lm_key_count + 1), 256);
    }
    l.total = off;
    return l;
}

}  // namespace ctcsd

using namespace ctcsd;

// The workspace size depends on the SM count only through upper bounds; 160 covers every
// B200 configuration and lets the size be queried without a device.
static const int kLayoutSms = 160;

extern "C" int ctcsd_workspace_bytes(const ctcsd_config* cfg, size_t* out_bytes) {
    if (!cfg || !out_bytes) return CTCSD_ERR_INVALID_ARG;
    int rc = validate_config(*cfg);
    if (rc != CTCSD_OK) return rc;
    *out_bytes = make_layout(*cfg, kLayoutSms).total;
    return CTCSD_OK;
}

extern "C" int ctcsd_create(ctcsd_handle** out_handle, const ctcsd_config* cfg, void* workspace, size_t workspace_bytes) {
    if (!out_handle || !cfg) return CTCSD_ERR_INVALID_ARG;
    *out_handle = nullptr;
    int rc = validate_config(*cfg);
    if (rc != CTCSD_OK) return rc;
    Layout lay = make_layout(*cfg, kLayoutSms);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) != 0 || workspace_bytes < lay.total)
        return CTCSD_ERR_WORKSPACE;
    ctcsd_handle* hh = new (std::nothrow) ctcsd_handle;
    if (!hh) return CTCSD_ERR_INTERNAL;
    Handle* h = &hh->h;
    memset(h, 0, sizeof(*h));
    h->cfg = *cfg;
    if (h->cfg.max_draft_rows == 0) h->cfg.max_draft_rows = cfg->B;
    h->lay = lay;
    h->ws = static_cast<char*>(workspace);
    cudaError_t e = cudaGetDevice(&h->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, h->device);
    int major = 0;
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, h->device);
    if (e == cudaSuccess && major != 10) { delete hh; return CTCSD_ERR_UNSUPPORTED; }
    if (e == cudaSuccess && h->num_sms > kLayoutSms) { delete hh; return CTCSD_ERR_UNSUPPORTED; }
    // status word, ticket counters and running maxima start at zero
    if (e == cudaSuccess) e = cudaMemset(workspace, 0, lay.zeroed_bytes);
    if (e != cudaSuccess) { delete hh; return CTCSD_ERR_CUDA; }
    *out_handle = hh;
    return CTCSD_OK;
}

extern "C" int ctcsd_destroy(ctcsd_handle* h) {
    if (!h) return CTCSD_ERR_INVALID_ARG;
    delete h;
    return CTCSD_OK;
}

extern "C" int ctcsd_poll_status(ctcsd_handle* hh, void* stream, int* out_status) {
    if (!hh || !out_status) return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int st[2] = {0, 0};
    CTCSD_CUDA_CHECK(h, cudaMemcpyAsync(st, status_ptr(h), sizeof(st), cudaMemcpyDeviceToHost, s));
    CTCSD_CUDA_CHECK(h, cudaStreamSynchronize(s));
    if (st[0] != 0) {
        // a kernel that gave up may have left its ticket counters and running maxima mid-way
        CTCSD_CUDA_CHECK(h, cudaMemsetAsync(h->ws, 0, h->lay.zeroed_bytes, s));
        CTCSD_CUDA_CHECK(h, cudaStreamSynchronize(s));
    }
    *out_status = st[0];
    return CTCSD_OK;
}

extern "C" int ctcsd_set_l2_prefetch(ctcsd_handle* hh, const void* ptr, size_t bytes) {
    if (!hh || (bytes != 0 && !ptr) || (reinterpret_cast<uintptr_t>(ptr) & 15)) return CTCSD_ERR_INVALID_ARG;
    hh->h.l2_hint_ptr = bytes ? ptr : nullptr;
    hh->h.l2_hint_bytes = bytes;
    return CTCSD_OK;
}

extern "C" const char* ctcsd_strerror(int status) {
    switch (status) {
        case CTCSD_OK: return "ok";
        case CTCSD_ERR_INVALID_ARG: return "invalid argument";
        case CTCSD_ERR_UNSUPPORTED: return "unsupported configuration";
        case CTCSD_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case CTCSD_ERR_CUDA: return "CUDA call failed";
        case CTCSD_ERR_TIMEOUT: return "device-side wait timed out";
        case CTCSD_ERR_INTERNAL: return "internal error";
        case CTCSD_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
        default: return "unknown status";
    }
}

extern "C" int ctcsd_debug_bounds_enabled(void) {
#ifdef CTCSD_DEBUG_BOUNDS
    return 1;
#else
    return 0;
#endif
}

extern "C" int ctcsd_last_cuda_error(const ctcsd_handle* h) { return h ? h->h.last_cuda_error : 0; }

extern "C" long long ctcsd_launch_count(const ctcsd_handle* h) { return h ? h->h.launches : 0; }

// ---------------------------------------------------------------------------------------
// Self-test of the bounded-wait machinery
// ---------------------------------------------------------------------------------------
#include "tc_primitives.cuh"

namespace ctcsd {
namespace {

// Waits on an mbarrier that nothing ever arrives on, with the same bounded wait the streaming
// kernels use but a short limit, and records the outcome the way they do.
__global__ void __launch_bounds__(32) selftest_timeout_kernel(int* status, long long limit_cycles) {
    __shared__ uint64_t bar;
    __shared__ int never_set;
    if (threadIdx.x == 0) {
        tc::mbar_init(&bar, 1);
        never_set = 0;
        tc::fence_barrier_init();
    }
    __syncwarp();
    if (threadIdx.x == 0) {
        const bool done = tc::mbar_wait(&bar, 0u, &never_set, limit_cycles);
        if (!done) report_error(status, CTCSD_ERR_TIMEOUT, 99);
    }
}

}  // namespace
}  // namespace ctcsd

extern "C" int ctcsd_selftest_timeout(ctcsd_handle* hh, void* stream) {
    if (!hh) return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    // about a millisecond at 2 GHz: long enough to be a real wait, short enough for a test
    selftest_timeout_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status_ptr(h), 2000000ll);
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}
