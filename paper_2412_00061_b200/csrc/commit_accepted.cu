// ctcsd_commit_accepted: after acceptance the accepted path becomes part of the cached prefix
// (paper Sec. 3.3, last paragraph: what a step outputs is appended to the history).
#include "common.cuh"

namespace ctcsd {
namespace {

struct CommitParams {
    void* K; void* V;                    // [B,Hkv,Lcap,D]
    const int* kv_len; const int* acc_len; const int* acc_nodes;
    int B, Hkv, Lcap, T, max_nodes, row_bytes;
    int* out_kv_len; int* out_sel_row;
    unsigned* seq_ticket;                // [B], zero between calls
    int* status;
};

// One CTA per (kv head, sequence).  Accepted node l sits at cache row L + node_l and belongs at
// row L + 1 + l.  Since node_l >= l + 1 a destination can be the source of an earlier accepted
// node, so all source rows go to shared memory first and are written back after a barrier.
__global__ void __launch_bounds__(256) commit_accepted_kernel(CommitParams p) {
    extern __shared__ __align__(16) unsigned char rows[];            // [2][T][row_bytes]
    const int g = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    pdl_wait();                          // the accepted path comes from the preceding kernel
    pdl_trigger();
    const int L = p.kv_len[b];
    int n = p.acc_len[b];
    const int chunks = p.row_bytes / 16;
    bool bad = n < 0 || n > p.T || L < 0 || L + 1 + n > p.Lcap;
    for (int l = 0; l < n && !bad; ++l) {
        const int node = p.acc_nodes[b * p.T + l];
        bad = node < l + 1 || node >= p.max_nodes || L + node >= p.Lcap;
    }
    if (bad) {                           // would read or write outside the cache: change nothing
        if (tid == 0) report_error(p.status, CTCSD_ERR_INVALID_ARG, b);
        n = 0;
    }
    unsigned char* Kb = static_cast<unsigned char*>(p.K) + ((size_t)b * p.Hkv + g) * (size_t)p.Lcap * p.row_bytes;
    unsigned char* Vb = static_cast<unsigned char*>(p.V) + ((size_t)b * p.Hkv + g) * (size_t)p.Lcap * p.row_bytes;
    for (int i = tid; i < 2 * n * chunks; i += blockDim.x) {
        const int which = i / (n * chunks), r = i - which * n * chunks;
        const int l = r / chunks, ch = r - l * chunks;
        const int node = p.acc_nodes[b * p.T + l];
        const unsigned char* src = (which ? Vb : Kb) + (size_t)(L + node) * p.row_bytes;
        reinterpret_cast<uint4*>(rows)[(which * p.T + l) * chunks + ch] = reinterpret_cast<const uint4*>(src)[ch];
    }
    __syncthreads();
    for (int i = tid; i < 2 * n * chunks; i += blockDim.x) {
        const int which = i / (n * chunks), r = i - which * n * chunks;
        const int l = r / chunks, ch = r - l * chunks;
        unsigned char* dst = (which ? Vb : Kb) + (size_t)(L + 1 + l) * p.row_bytes;
        reinterpret_cast<uint4*>(dst)[ch] = reinterpret_cast<const uint4*>(rows)[(which * p.T + l) * chunks + ch];
    }
    // out_kv_len may be the very array kv_len: the new length is written by whichever CTA of the
    // sequence finishes last, when every kv head's CTA has read the old one
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        if (atomicAdd(&p.seq_ticket[b], 1u) == (unsigned)p.Hkv - 1u) {
            p.seq_ticket[b] = 0u;
            p.out_kv_len[b] = bad ? L : L + 1 + n;
            if (p.out_sel_row) p.out_sel_row[b] = b * p.max_nodes + (n > 0 ? p.acc_nodes[b * p.T + n - 1] : 0);
        }
    }
}

}  // namespace
}  // namespace ctcsd

using namespace ctcsd;

extern "C" int ctcsd_commit_accepted(ctcsd_handle* hh, void* stream, void* K, void* V, int Lcap,
                                     const int* kv_len, const int* acc_len, const int* acc_nodes,
                                     int* out_kv_len, int* out_sel_row) {
    if (!hh || !K || !V || !kv_len || !acc_len || !acc_nodes || !out_kv_len) return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    const ctcsd_config& c = h->cfg;
    if (Lcap < c.max_nodes) return CTCSD_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V)) & 15) return CTCSD_ERR_INVALID_ARG;
    CommitParams p;
    p.K = K; p.V = V;
    p.kv_len = kv_len; p.acc_len = acc_len; p.acc_nodes = acc_nodes;
    p.B = c.B; p.Hkv = c.Hkv; p.Lcap = Lcap; p.T = c.T; p.max_nodes = c.max_nodes;
    p.row_bytes = c.D * (c.dtype == CTCSD_DTYPE_BF16 ? 2 : 4);
    p.out_kv_len = out_kv_len; p.out_sel_row = out_sel_row;
    p.status = status_ptr(h);
    p.seq_ticket = reinterpret_cast<unsigned*>(h->ws + h->lay.seq_ticket_off);
    const size_t smem = (size_t)2 * c.T * p.row_bytes;
    CTCSD_CUDA_CHECK(h, launch_pdl(commit_accepted_kernel, dim3(c.Hkv, c.B), dim3(256), smem,
                                   static_cast<cudaStream_t>(stream), 1, p));
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}
