// ctcsd_tree_attention_static: tree attention for callers that cannot allocate device memory.
//
// The regular entry point keeps the per-split partial results (running max, sum and
// unnormalised output of every KV split) in the workspace that the caller allocated for its
// handle.  A caller that lives inside somebody else's memory plan - a plug-in that is handed
// its tensors by a runtime and may not call cudaMalloc, code running where the allocator is
// frozen after start-up, a real-time loop in which an allocation could stall the device - has
// no such workspace to give.  For them the partials live in a fixed array that is part of
// this library's device image, so nothing is allocated, by this library or by CUDA on its
// behalf, when the call is made.
#include "tree_attention.cuh"

#include <mutex>

namespace ctcsd {
namespace {

// 32 MiB of partials + one 256-byte block for the status word.  Every device that loads the
// library keeps this much memory reserved until the process exits.
constexpr size_t kStaticPartBytes = (size_t)CTCSD_STATIC_ATTN_SCRATCH_BYTES;
constexpr size_t kStaticHeadBytes = 256;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticHeadBytes + kStaticPartBytes];

constexpr int kMaxDevices = 64;
struct DeviceSetup {
    bool ready;
    unsigned char* scratch;     // device address of g_static_scratch on this device
    int num_sms;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_mutex;

// First call on a device: resolve the array's device address.  In host code the array's name
// only stands for the symbol; the address a kernel can use has to be asked for, with the
// device in question current (it is: the entry point works on the current device).
int setup_current_device(DeviceSetup** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return CTCSD_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return CTCSD_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    DeviceSetup& d = g_setup[dev];
    if (!d.ready) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) return CTCSD_ERR_CUDA;
        int sms = 0, major = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return CTCSD_ERR_CUDA;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return CTCSD_ERR_CUDA;
        if (major != 10) return CTCSD_ERR_UNSUPPORTED;
        d.scratch = static_cast<unsigned char*>(ptr);
        d.num_sms = sms;
        d.ready = true;
    }
    *out = &d;
    return CTCSD_OK;
}

}  // namespace
}  // namespace ctcsd

using namespace ctcsd;

extern "C" int ctcsd_tree_attention_static(void* stream, int B, int max_nodes, int Hq, int Hkv, int D,
                                           const void* Q, const void* K, const void* V, int Lcap,
                                           const int* kv_len, const int* n_nodes,
                                           const unsigned long long* mask, float scale, void* out_O,
                                           int* out_status) {
    if (!Q || !K || !V || !kv_len || !n_nodes || !mask || !out_O) return CTCSD_ERR_INVALID_ARG;
    if (B < 1 || max_nodes < 2 || max_nodes > 128) return CTCSD_ERR_INVALID_ARG;
    if (Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || (D != 64 && D != 128)) return CTCSD_ERR_INVALID_ARG;
    if (Lcap < max_nodes || (long long)B * max_nodes > (1 << 20)) return CTCSD_ERR_INVALID_ARG;

    const size_t per_split = (size_t)B * Hq * max_nodes * (D + 2) * sizeof(float);
    if (per_split > kStaticPartBytes) return CTCSD_ERR_TOO_LARGE;

    DeviceSetup* dev = nullptr;
    int rc = setup_current_device(&dev);
    if (rc != CTCSD_OK) return rc;

    // as many KV splits as keep two CTAs per SM busy, fewer if the partials would not fit
    const long long units = (long long)B * Hkv;
    long long splits = (2ll * dev->num_sms + units - 1) / units;
    if (splits > 16) splits = 16;
    if ((size_t)splits * per_split > kStaticPartBytes) splits = (long long)(kStaticPartBytes / per_split);
    if (splits < 1) splits = 1;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    AttnParams p;
    p.Q = Q; p.K = K; p.V = V; p.O = out_O;
    p.kv_len = kv_len; p.n_nodes = n_nodes; p.mask = mask;
    p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.D = D; p.max_nodes = max_nodes; p.Lcap = Lcap;
    p.scale = scale;
    // the status word has to start at zero; the partials need no clearing (every entry that the
    // merge reads is written by this call first)
    int* status = out_status ? out_status : reinterpret_cast<int*>(dev->scratch);
    if (cudaMemsetAsync(status, 0, 2 * sizeof(int), s) != cudaSuccess) return CTCSD_ERR_CUDA;
    p.status = status;
    float* part = reinterpret_cast<float*>(dev->scratch + kStaticHeadBytes);
    if (launch_tree_attention_mma_scratch(s, p, part, (int)splits) != cudaSuccess) return CTCSD_ERR_CUDA;
    return CTCSD_OK;
}
