// ctcsd_draft_module: the paper's Attention Draft Module (Sec. 3.1: one transformer layer, built
// like the base model's layers, on the base model's hidden states; Sec. 3.2: F_hat =
// DraftModule(F), which the per-place projection then turns into one distribution per place).
//
// The layer is a LLaMA-style decoder layer: RMSNorm, rotary self-attention over the hidden states
// of all positions so far (keys/values of earlier positions cached), residual, RMSNorm, SwiGLU
// MLP, residual.  Per decoding step it sees the hidden states of the few newest positions of every
// sequence; keys/values are made for all of them, the rest of the layer runs for the newest one
// only, whose output is the state the draft head projects.  At batch 1 every projection is a
// matrix-vector product bound by HBM: the four weight matrices go through the same
// weight-streaming kernel as the draft head (plain-output mode); the attention is the
// tree-attention kernel on a one-node tree; the pieces between them are row-sized kernels.
#include "gemv_stream.cuh"
#include "tree_attention.cuh"

#include <math.h>
#include <string.h>

namespace ctcsd {

int tree_attention_dispatch(Handle* h, cudaStream_t s, const AttnParams& p);

namespace {

template <typename T> __device__ __forceinline__ float ld_f(const T* p, size_t i);
template <> __device__ __forceinline__ float ld_f<float>(const float* p, size_t i) { return p[i]; }
template <> __device__ __forceinline__ float ld_f<__nv_bfloat16>(const __nv_bfloat16* p, size_t i) { return __bfloat162float(p[i]); }
template <typename T> __device__ __forceinline__ void st_f(T* p, size_t i, float v);
template <> __device__ __forceinline__ void st_f<float>(float* p, size_t i, float v) { p[i] = v; }
template <> __device__ __forceinline__ void st_f<__nv_bfloat16>(__nv_bfloat16* p, size_t i, float v) { p[i] = __float2bfloat16_rn(v); }

__device__ __forceinline__ float block_sum(float v, float* red) {
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
    return t;
}

struct DmParams {
    const void* F_new;          // [B,R,H] act dtype
    const int* n_new;           // [B]
    const int* kv_len;          // [B] positions already in the layer's cache
    void* Kd; void* Vd;         // [B,Hkv,Lcap,D] act dtype
    const float* g1; const float* g2;
    int B, R, H, Hq, Hkv, D, I, Lcap, max_nodes;
    float eps, theta;
    // scratch
    void* a;                    // [B*R,H] act: normalised new rows
    float* qkv;                 // [B*R,(Hq+2Hkv)D]
    void* Qbuf;                 // [B,max_nodes,Hq,D] act: node 0 holds the newest position's query
    void* Obuf;                 // [B,max_nodes,Hq,D] act
    int* attn_len;              // [B] keys before the query row = kv_len + n_new - 1
    int* ones;                  // [B] = 1
    int* o_rows;                // [B] = b * max_nodes
    unsigned long long* mask;   // [B,max_nodes,W], bit 0 of row 0 set
    float* o;                   // [B,H] attention output projection
    float* h1;                  // [B,H] after the first residual
    void* m;                    // [B,H] act: normalised h1
    float* gu;                  // [B,2I]
    void* act;                  // [B,I] act: SiLU(gate) * up
    float* mlp;                 // [B,H]
    void* out_F;                // [B,H] act
    float* out_F_dbg;           // null or [B,H]
    int* out_kv_len;            // [B]
    int* status;
};

// RMSNorm of every new row; rows past n_new[b] are written as zero.  One CTA per (row j, sequence b).
template <typename T>
__global__ void __launch_bounds__(256) dm_norm_rows_kernel(DmParams p) {
    __shared__ float red[8];
    const int j = blockIdx.x, b = blockIdx.y;
    pdl_wait();
    pdl_trigger();
    const T* src = static_cast<const T*>(p.F_new) + ((size_t)b * p.R + j) * p.H;
    T* dst = static_cast<T*>(p.a) + ((size_t)b * p.R + j) * p.H;
    int r = p.n_new[b];
    r = r < 0 ? 0 : (r > p.R ? p.R : r);
    if (j >= r) {
        for (int i = threadIdx.x; i < p.H; i += blockDim.x) st_f<T>(dst, i, 0.f);
        return;
    }
    float ss = 0.f;
    for (int i = threadIdx.x; i < p.H; i += blockDim.x) { const float v = ld_f<T>(src, i); ss += v * v; }
    ss = block_sum(ss, red);
    const float inv = rsqrtf(ss / (float)p.H + p.eps);
    for (int i = threadIdx.x; i < p.H; i += blockDim.x) st_f<T>(dst, i, ld_f<T>(src, i) * inv * p.g1[i]);
}

// Rotary embedding and placement: keys/values of every new position go to the layer's cache, the
// newest position's query to node 0 of the query buffer; also fills the small arrays that describe
// the one-node "tree" to the attention kernel.  One CTA per (row j, sequence b); thread = (head, pair).
template <typename T>
__global__ void __launch_bounds__(256) dm_rope_scatter_kernel(DmParams p) {
    const int j = blockIdx.x, b = blockIdx.y;
    pdl_wait();
    pdl_trigger();
    const int L = p.kv_len[b];
    int r = p.n_new[b];
    const bool bad = r < 1 || r > p.R || L < 0 || L + r > p.Lcap;
    if (bad) r = 0;
    const int W = (p.max_nodes + 63) / 64;
    if (j == 0) {
        if (threadIdx.x == 0) {
            if (bad) report_error(p.status, CTCSD_ERR_INVALID_ARG, b);
            p.attn_len[b] = bad ? 0 : L + r - 1;
            p.ones[b] = bad ? 0 : 1;
            p.o_rows[b] = b * p.max_nodes;
            p.out_kv_len[b] = bad ? L : L + r;
        }
        for (int i = threadIdx.x; i < p.max_nodes * W; i += blockDim.x)
            p.mask[(size_t)b * p.max_nodes * W + i] = (i == 0) ? 1ull : 0ull;
    }
    if (j >= r) return;
    const int half = p.D / 2, Nq = p.Hq * p.D, Nk = p.Hkv * p.D;
    const float* row = p.qkv + ((size_t)b * p.R + j) * (size_t)(Nq + 2 * Nk);
    const int pos = L + j;
    const bool newest = (j == r - 1);
    T* Kd = static_cast<T*>(p.Kd);
    T* Vd = static_cast<T*>(p.Vd);
    T* Qb = static_cast<T*>(p.Qbuf);
    const int heads = p.Hq + p.Hkv;                       // rotated heads: queries then keys
    for (int w = threadIdx.x; w < heads * half; w += blockDim.x) {
        const int hd = w / half, i = w - hd * half;
        const bool is_q = hd < p.Hq;
        if (is_q && !newest) continue;
        const float* v = row + (is_q ? hd * p.D : Nq + (hd - p.Hq) * p.D);
        // angle = pos * theta^(-2i/D), formed in float64 so that long positions keep their phase
        const double ang = (double)pos * exp2(-2.0 * (double)i / (double)p.D * log2((double)p.theta));
        float sn, cs;
        sincosf((float)fmod(ang, 6.283185307179586476925286766559), &sn, &cs);
        const float x0 = v[i], x1 = v[i + half];
        const float y0 = x0 * cs - x1 * sn, y1 = x1 * cs + x0 * sn;
        if (is_q) {
            T* dst = Qb + (((size_t)b * p.max_nodes + 0) * p.Hq + hd) * p.D;
            st_f<T>(dst, i, y0);
            st_f<T>(dst, i + half, y1);
        } else {
            T* dst = Kd + (((size_t)b * p.Hkv + (hd - p.Hq)) * p.Lcap + pos) * p.D;
            st_f<T>(dst, i, y0);
            st_f<T>(dst, i + half, y1);
        }
    }
    for (int w = threadIdx.x; w < Nk; w += blockDim.x) {
        const int g = w / p.D, d = w - g * p.D;
        st_f<T>(Vd + (((size_t)b * p.Hkv + g) * p.Lcap + pos) * p.D, d, row[Nq + Nk + w]);
    }
}

// h1 = F_last + o;  m = RMSNorm(h1) * g2.  One CTA per sequence.
template <typename T>
__global__ void __launch_bounds__(256) dm_residual_norm_kernel(DmParams p) {
    __shared__ float red[8];
    const int b = blockIdx.x;
    pdl_wait();
    pdl_trigger();
    int r = p.n_new[b];
    r = r < 1 ? 1 : (r > p.R ? p.R : r);
    const T* src = static_cast<const T*>(p.F_new) + ((size_t)b * p.R + (r - 1)) * p.H;
    float* h1 = p.h1 + (size_t)b * p.H;
    float ss = 0.f;
    for (int i = threadIdx.x; i < p.H; i += blockDim.x) {
        const float v = ld_f<T>(src, i) + p.o[(size_t)b * p.H + i];
        h1[i] = v;
        ss += v * v;
    }
    ss = block_sum(ss, red);
    const float inv = rsqrtf(ss / (float)p.H + p.eps);
    T* dst = static_cast<T*>(p.m) + (size_t)b * p.H;
    for (int i = threadIdx.x; i < p.H; i += blockDim.x) st_f<T>(dst, i, h1[i] * inv * p.g2[i]);
}

// act = SiLU(gate) * up
template <typename T>
__global__ void __launch_bounds__(256) dm_swiglu_kernel(DmParams p) {
    pdl_wait();
    pdl_trigger();
    const size_t n = (size_t)p.B * p.I;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const size_t b = e / p.I, i = e - b * p.I;
        const float g = p.gu[b * 2 * p.I + i], u = p.gu[b * 2 * p.I + p.I + i];
        st_f<T>(static_cast<T*>(p.act), e, g / (1.f + __expf(-g)) * u);
    }
}

// F_hat = h1 + mlp
template <typename T>
__global__ void __launch_bounds__(256) dm_residual_out_kernel(DmParams p) {
    pdl_wait();
    pdl_trigger();
    const size_t n = (size_t)p.B * p.H;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (size_t)gridDim.x * blockDim.x) {
        const float v = p.h1[e] + p.mlp[e];
        st_f<T>(static_cast<T*>(p.out_F), e, v);
        if (p.out_F_dbg) p.out_F_dbg[e] = v;
    }
}

struct DmLayout {
    size_t a, qkv, Qbuf, Obuf, attn_len, ones, o_rows, mask, o, h1, m, gu, act, mlp, total;
};

DmLayout dm_layout(const ctcsd_config& c, int R, int I) {
    DmLayout l;
    const size_t esz = c.dtype == CTCSD_DTYPE_BF16 ? 2 : 4;
    const size_t W = (c.max_nodes + 63) / 64;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return at; };
    l.a = take((size_t)c.B * R * c.H * esz);
    l.qkv = take((size_t)c.B * R * (c.Hq + 2 * c.Hkv) * c.D * 4);
    l.Qbuf = take((size_t)c.B * c.max_nodes * c.Hq * c.D * esz);
    l.Obuf = take((size_t)c.B * c.max_nodes * c.Hq * c.D * esz);
    l.attn_len = take((size_t)c.B * 4);
    l.ones = take((size_t)c.B * 4);
    l.o_rows = take((size_t)c.B * 4);
    l.mask = take((size_t)c.B * c.max_nodes * W * 8);
    l.o = take((size_t)c.B * c.H * 4);
    l.h1 = take((size_t)c.B * c.H * 4);
    l.m = take((size_t)c.B * c.H * esz);
    l.gu = take((size_t)c.B * 2 * I * 4);
    l.act = take((size_t)c.B * I * esz);
    l.mlp = take((size_t)c.B * c.H * 4);
    l.total = off;
    return l;
}

// y[M,N] = x[rows picked by x_rows][K] . W[N,K]^T as float32, through the weight-streaming kernel.
int plain_gemv(Handle* h, cudaStream_t s, int M, const void* x, int x_row_count, const int* x_rows, const void* W,
               int K, int N, float* y) {
    GemvParams g;
    memset(&g, 0, sizeof(g));
    g.x = x; g.x_rows = x_rows; g.x_row_count = x_row_count; g.W = W;
    g.H = K; g.slots = 1; g.rows_per_slot = N;
    g.mode = 2; g.k = 1;
    g.logits_dbg = y;
    g.sn.max_nodes = 1; g.sn.rows_per_seq = 1; g.sn.inv_temp = 1.f;
    return launch_gemv_stream(h, s, h->cfg.dtype, M, g);
}

template <typename T>
int run_draft_module(Handle* h, cudaStream_t s, DmParams& p, const void* Wqkv, const void* Wo, const void* Wgu,
                     const void* Wdn) {
    const ctcsd_config& c = h->cfg;
    CTCSD_CUDA_CHECK(h, launch_pdl(dm_norm_rows_kernel<T>, dim3(p.R, p.B), dim3(256), 0, s, 1, p));
    CTCSD_LAUNCH_CHECK(h);
    const int Nqkv = (c.Hq + 2 * c.Hkv) * c.D;
    int rc = plain_gemv(h, s, p.B * p.R, p.a, p.B * p.R, nullptr, Wqkv, c.H, Nqkv, p.qkv);
    if (rc != CTCSD_OK) return rc;
    CTCSD_CUDA_CHECK(h, launch_pdl(dm_rope_scatter_kernel<T>, dim3(p.R, p.B), dim3(256), 0, s, 1, p));
    CTCSD_LAUNCH_CHECK(h);
    AttnParams ap;
    ap.Q = p.Qbuf; ap.K = p.Kd; ap.V = p.Vd; ap.O = p.Obuf;
    ap.kv_len = p.attn_len; ap.n_nodes = p.ones; ap.mask = p.mask;
    ap.B = c.B; ap.Hq = c.Hq; ap.Hkv = c.Hkv; ap.D = c.D; ap.max_nodes = c.max_nodes; ap.Lcap = p.Lcap;
    ap.scale = 1.0f / sqrtf((float)c.D);
    ap.status = p.status;
    rc = tree_attention_dispatch(h, s, ap);
    if (rc != CTCSD_OK) return rc;
    rc = plain_gemv(h, s, p.B, p.Obuf, p.B * c.max_nodes, p.o_rows, Wo, c.Hq * c.D, c.H, p.o);
    if (rc != CTCSD_OK) return rc;
    CTCSD_CUDA_CHECK(h, launch_pdl(dm_residual_norm_kernel<T>, dim3(p.B), dim3(256), 0, s, 1, p));
    CTCSD_LAUNCH_CHECK(h);
    rc = plain_gemv(h, s, p.B, p.m, p.B, nullptr, Wgu, c.H, 2 * p.I, p.gu);
    if (rc != CTCSD_OK) return rc;
    const int eb = (int)(((size_t)p.B * p.I + 255) / 256);
    CTCSD_CUDA_CHECK(h, launch_pdl(dm_swiglu_kernel<T>, dim3(eb < 1184 ? eb : 1184), dim3(256), 0, s, 1, p));
    CTCSD_LAUNCH_CHECK(h);
    rc = plain_gemv(h, s, p.B, p.act, p.B, nullptr, Wdn, p.I, c.H, p.mlp);
    if (rc != CTCSD_OK) return rc;
    const int ob = (int)(((size_t)p.B * p.H + 255) / 256);
    CTCSD_CUDA_CHECK(h, launch_pdl(dm_residual_out_kernel<T>, dim3(ob < 1184 ? ob : 1184), dim3(256), 0, s, 1, p));
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}

}  // namespace
}  // namespace ctcsd

using namespace ctcsd;

extern "C" int ctcsd_draft_module_workspace_bytes(const ctcsd_config* cfg, int R, int I, size_t* out_bytes) {
    if (!cfg || !out_bytes || R < 1 || R > CTCSD_MAX_T + 1 || I < 8 || I % 8 != 0) return CTCSD_ERR_INVALID_ARG;
    int rc = validate_config(*cfg);
    if (rc != CTCSD_OK) return rc;
    *out_bytes = dm_layout(*cfg, R, I).total;
    return CTCSD_OK;
}

extern "C" int ctcsd_draft_module(ctcsd_handle* hh, void* stream, const ctcsd_draft_layer* layer,
                                  void* workspace, size_t workspace_bytes,
                                  int R, const void* F_new, const int* n_new, const int* kv_len,
                                  void* Kd, void* Vd, int Lcap,
                                  void* out_F, int* out_kv_len, float* out_F_dbg) {
    if (!hh || !layer || !workspace || !F_new || !n_new || !kv_len || !Kd || !Vd || !out_F || !out_kv_len)
        return CTCSD_ERR_INVALID_ARG;
    if (!layer->g1 || !layer->Wqkv || !layer->Wo || !layer->g2 || !layer->Wgu || !layer->Wdn) return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    const ctcsd_config& c = h->cfg;
    const int I = layer->I;
    if (R < 1 || R > CTCSD_MAX_T + 1 || I < 8 || I % 8 != 0 || Lcap < 1 || (c.D & 1)) return CTCSD_ERR_INVALID_ARG;
    if (!(layer->eps > 0.f) || !(layer->rope_theta > 1.f)) return CTCSD_ERR_INVALID_ARG;
    const uintptr_t al = reinterpret_cast<uintptr_t>(F_new) | reinterpret_cast<uintptr_t>(Kd) | reinterpret_cast<uintptr_t>(Vd) |
                         reinterpret_cast<uintptr_t>(layer->Wqkv) | reinterpret_cast<uintptr_t>(layer->Wo) |
                         reinterpret_cast<uintptr_t>(layer->Wgu) | reinterpret_cast<uintptr_t>(layer->Wdn);
    if (al & 15) return CTCSD_ERR_INVALID_ARG;
    const DmLayout l = dm_layout(c, R, I);
    if ((reinterpret_cast<uintptr_t>(workspace) & 255) != 0 || workspace_bytes < l.total) return CTCSD_ERR_WORKSPACE;
    char* ws = static_cast<char*>(workspace);
    DmParams p;
    memset(&p, 0, sizeof(p));
    p.F_new = F_new; p.n_new = n_new; p.kv_len = kv_len; p.Kd = Kd; p.Vd = Vd;
    p.g1 = layer->g1; p.g2 = layer->g2;
    p.B = c.B; p.R = R; p.H = c.H; p.Hq = c.Hq; p.Hkv = c.Hkv; p.D = c.D; p.I = I; p.Lcap = Lcap; p.max_nodes = c.max_nodes;
    p.eps = layer->eps; p.theta = layer->rope_theta;
    p.a = ws + l.a; p.qkv = reinterpret_cast<float*>(ws + l.qkv);
    p.Qbuf = ws + l.Qbuf; p.Obuf = ws + l.Obuf;
    p.attn_len = reinterpret_cast<int*>(ws + l.attn_len); p.ones = reinterpret_cast<int*>(ws + l.ones);
    p.o_rows = reinterpret_cast<int*>(ws + l.o_rows); p.mask = reinterpret_cast<unsigned long long*>(ws + l.mask);
    p.o = reinterpret_cast<float*>(ws + l.o); p.h1 = reinterpret_cast<float*>(ws + l.h1); p.m = ws + l.m;
    p.gu = reinterpret_cast<float*>(ws + l.gu); p.act = ws + l.act; p.mlp = reinterpret_cast<float*>(ws + l.mlp);
    p.out_F = out_F; p.out_F_dbg = out_F_dbg; p.out_kv_len = out_kv_len;
    p.status = status_ptr(h);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (c.dtype == CTCSD_DTYPE_BF16)
        return run_draft_module<__nv_bfloat16>(h, s, p, layer->Wqkv, layer->Wo, layer->Wgu, layer->Wdn);
    return run_draft_module<float>(h, s, p, layer->Wqkv, layer->Wo, layer->Wgu, layer->Wdn);
}
