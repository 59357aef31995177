// ctcsd_tree_attention: softmax(q k^T * scale) v over the cached prefix plus the tree
// nodes allowed by the ancestor mask.
#include "tree_attention.cuh"

#include <math.h>

namespace ctcsd {
namespace {

// ---------------------------------------------------------------------------------------
// Reference-grade kernel for any dtype: one CTA per (node, head, sequence); its four warps
// stride over the keys, every lane owning D/32 dimensions, each warp keeping an online
// softmax state that is merged through shared memory at the end.
// ---------------------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T, int D>
__global__ void __launch_bounds__(128) tree_attention_simple_kernel(AttnParams p) {
    constexpr int PER = D / 32;
    const int i = blockIdx.x, hq = blockIdx.y, b = blockIdx.z;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int n = p.n_nodes[b];
    const int L = p.kv_len[b];
    T* out = reinterpret_cast<T*>(p.O) + (((size_t)b * p.max_nodes + i) * p.Hq + hq) * D;
    if (n < 0 || n > p.max_nodes || L < 0 || L + n > p.Lcap) {       // would read outside the cache
        if (threadIdx.x == 0) report_error(p.status, CTCSD_ERR_INVALID_ARG, b);
        n = 0;
    }
    if (i >= n) {
        if (warp == 0)
            for (int d = 0; d < PER; ++d) out[lane + 32 * d] = from_f<T>(0.f);
        return;
    }
    const int hk = hq / (p.Hq / p.Hkv);
    const T* q = reinterpret_cast<const T*>(p.Q) + (((size_t)b * p.max_nodes + i) * p.Hq + hq) * D;
    const T* Kb = reinterpret_cast<const T*>(p.K) + ((size_t)b * p.Hkv + hk) * (size_t)p.Lcap * D;
    const T* Vb = reinterpret_cast<const T*>(p.V) + ((size_t)b * p.Hkv + hk) * (size_t)p.Lcap * D;
    const int W = (p.max_nodes + 63) / 64;
    const unsigned long long* mrow = p.mask + ((size_t)b * p.max_nodes + i) * W;

    float qv[PER], acc[PER];
#pragma unroll
    for (int d = 0; d < PER; ++d) { qv[d] = to_f<T>(q[lane + 32 * d]) * p.scale; acc[d] = 0.f; }
    float mx = -INFINITY, sum = 0.f;
    for (int j = warp; j < L + n; j += 4) {
        if (j >= L) {
            int t = j - L;
            if (!((mrow[t >> 6] >> (t & 63)) & 1ull)) continue;
        }
        const T* kr = Kb + (size_t)j * D;
        float s = 0.f;
#pragma unroll
        for (int d = 0; d < PER; ++d) s = fmaf(qv[d], to_f<T>(kr[lane + 32 * d]), s);
        s = warp_sum(s);
        float nm = fmaxf(mx, s);
        float corr = __expf(mx - nm), pj = __expf(s - nm);
        sum = sum * corr + pj;
        const T* vr = Vb + (size_t)j * D;
#pragma unroll
        for (int d = 0; d < PER; ++d) acc[d] = acc[d] * corr + pj * to_f<T>(vr[lane + 32 * d]);
        mx = nm;
    }
    __shared__ float s_mx[4], s_sum[4], s_acc[4][D];
    if (lane == 0) { s_mx[warp] = mx; s_sum[warp] = sum; }
#pragma unroll
    for (int d = 0; d < PER; ++d) s_acc[warp][lane + 32 * d] = acc[d];
    __syncthreads();
    if (warp == 0) {
        float gm = fmaxf(fmaxf(s_mx[0], s_mx[1]), fmaxf(s_mx[2], s_mx[3]));
        float tot = 0.f, o[PER];
#pragma unroll
        for (int d = 0; d < PER; ++d) o[d] = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            float f = (s_mx[w] == -INFINITY) ? 0.f : __expf(s_mx[w] - gm);
            tot += s_sum[w] * f;
#pragma unroll
            for (int d = 0; d < PER; ++d) o[d] += s_acc[w][lane + 32 * d] * f;
        }
        float inv = 1.f / tot;
#pragma unroll
        for (int d = 0; d < PER; ++d) out[lane + 32 * d] = from_f<T>(o[d] * inv);
    }
}

template <typename T>
int launch_simple(Handle* h, cudaStream_t s, const AttnParams& p) {
    dim3 grid(p.max_nodes, p.Hq, p.B);
    if (p.D == 64) tree_attention_simple_kernel<T, 64><<<grid, 128, 0, s>>>(p);
    else tree_attention_simple_kernel<T, 128><<<grid, 128, 0, s>>>(p);
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}

}  // namespace
}  // namespace ctcsd

namespace ctcsd {
// The attention kernel that serves the handle's dtype and head grouping.
int tree_attention_dispatch(Handle* h, cudaStream_t s, const AttnParams& p) {
    if (h->cfg.dtype == CTCSD_DTYPE_BF16) {
        if (tree_attention_tc_supported(p)) return launch_tree_attention_tc(h, s, p);
        return launch_tree_attention_mma(h, s, p);
    }
    return launch_simple<float>(h, s, p);
}
}  // namespace ctcsd

using namespace ctcsd;

extern "C" int ctcsd_tree_attention(ctcsd_handle* hh, void* stream, const void* Q, const void* K, const void* V,
                                    int Lcap, const int* kv_len, const int* n_nodes,
                                    const unsigned long long* mask, float scale, void* out_O) {
    if (!hh || !Q || !K || !V || !kv_len || !n_nodes || !mask || !out_O) return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    const ctcsd_config& c = h->cfg;
    if (Lcap < c.max_nodes) return CTCSD_ERR_INVALID_ARG;
    AttnParams p;
    p.Q = Q; p.K = K; p.V = V; p.O = out_O;
    p.kv_len = kv_len; p.n_nodes = n_nodes; p.mask = mask;
    p.B = c.B; p.Hq = c.Hq; p.Hkv = c.Hkv; p.D = c.D; p.max_nodes = c.max_nodes; p.Lcap = Lcap;
    p.scale = scale;
    p.status = status_ptr(h);
    return tree_attention_dispatch(h, static_cast<cudaStream_t>(stream), p);
}
