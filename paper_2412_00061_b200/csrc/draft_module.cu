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
// tree-attention kernel on a one-node tree.  The row-sized pieces between them ride along: both
// RMSNorms (the second with its residual) and the SwiGLU are applied by the projection that
// follows them while it loads its activation rows, the last residual by the projection before
// it as it writes its result; only the rotary embedding with the K/V append is a kernel of its
// own.  Six launches in all.
#include "gemv_stream.cuh"
#include "tree_attention.cuh"

#include <math.h>
#include <string.h>

namespace ctcsd {

int tree_attention_dispatch(Handle* h, cudaStream_t s, const AttnParams& p);

namespace {

template <typename T> __device__ __forceinline__ void st_f(T* p, size_t i, float v);
template <> __device__ __forceinline__ void st_f<float>(float* p, size_t i, float v) { p[i] = v; }
template <> __device__ __forceinline__ void st_f<__nv_bfloat16>(__nv_bfloat16* p, size_t i, float v) { p[i] = __float2bfloat16_rn(v); }

struct DmParams {
    const void* F_new;          // [B,R,H] act dtype
    const int* n_new;           // [B]
    const int* kv_len;          // [B] positions already in the layer's cache
    void* Kd; void* Vd;         // [B,Hkv,Lcap,D] act dtype
    const float* g1; const float* g2;
    int B, R, H, Hq, Hkv, D, I, Lcap, max_nodes;
    float eps, theta;
    double inv_freq[64];        // theta^(-2i/D), i < D/2, formed on the host in float64
    // scratch
    float* qkv;                 // [B*R,(Hq+2Hkv)D]
    void* Qbuf;                 // [B,max_nodes,Hq,D] act: node 0 holds the newest position's query
    void* Obuf;                 // [B,max_nodes,Hq,D] act
    int* attn_len;              // [B] keys before the query row = kv_len + n_new - 1
    int* ones;                  // [B] = 1
    int* o_rows;                // [B] = b * max_nodes
    int* last_rows;             // [B] = b * R + n_new[b] - 1: the newest position's row of F_new
    unsigned long long* mask;   // [B,max_nodes,W], bit 0 of row 0 set
    float* o;                   // [B,H] attention output projection
    float* h1;                  // [B,H] after the first residual
    float* gu;                  // [B,2I]
    void* out_F;                // [B,H] act
    float* out_F_dbg;           // null or [B,H]
    int* out_kv_len;            // [B]
    int* status;
};

// Rotary embedding and placement: keys/values of every new position go to the layer's cache, the
// newest position's query to node 0 of the query buffer; also fills the small arrays that describe
// the one-node "tree" to the attention kernel.  Eight CTAs per (row j, sequence b); thread = (head, pair).
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
    if (j == 0 && blockIdx.z == 0) {
        if (threadIdx.x == 0) {
            if (bad) report_error(p.status, CTCSD_ERR_INVALID_ARG, b);
            p.attn_len[b] = bad ? 0 : L + r - 1;
            p.ones[b] = bad ? 0 : 1;
            p.o_rows[b] = b * p.max_nodes;
            p.last_rows[b] = b * p.R + (bad ? 0 : r - 1);
            p.out_kv_len[b] = bad ? L : L + r;
        }
        for (int i = threadIdx.x; i < p.max_nodes * W; i += blockDim.x)
            p.mask[(size_t)b * p.max_nodes * W + i] = (i == 0) ? 1ull : 0ull;
    }
    if (j >= r) return;
    const int half = p.D / 2, Nq = p.Hq * p.D, Nk = p.Hkv * p.D;
    // the position is the CTA's: one sine and cosine per pair index, shared by all heads
    // (angle = pos * theta^(-2i/D), formed and reduced in float64 so that long positions keep their phase)
    __shared__ float s_sin[64], s_cos[64];                  // D is 64 or 128
    for (int i = threadIdx.x; i < half; i += blockDim.x) {
        const double two_pi = 6.283185307179586476925286766559;
        const double ang = (double)(L + j) * p.inv_freq[i];
        sincosf((float)(ang - floor(ang / two_pi) * two_pi), &s_sin[i], &s_cos[i]);   // reduced in float64, then float32
    }
    __syncthreads();
    const float* row = p.qkv + ((size_t)b * p.R + j) * (size_t)(Nq + 2 * Nk);
    const int pos = L + j;
    const bool newest = (j == r - 1);
    T* Kd = static_cast<T*>(p.Kd);
    T* Vd = static_cast<T*>(p.Vd);
    T* Qb = static_cast<T*>(p.Qbuf);
    const int heads = p.Hq + p.Hkv;                       // rotated heads: queries then keys
    // (the loops are chains of dependent loads from L2: the work of a row is spread over gridDim.z CTAs)
    const int tz = blockIdx.z * blockDim.x + threadIdx.x, nz = gridDim.z * blockDim.x;
    for (int w = tz; w < heads * half; w += nz) {
        const int hd = w / half, i = w - hd * half;
        const bool is_q = hd < p.Hq;
        if (is_q && !newest) continue;
        const float* v = row + (is_q ? hd * p.D : Nq + (hd - p.Hq) * p.D);
        const float sn = s_sin[i], cs = s_cos[i];
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
    for (int w = tz; w < Nk; w += nz) {
        const int g = w / p.D, d = w - g * p.D;
        st_f<T>(Vd + (((size_t)b * p.Hkv + g) * p.Lcap + pos) * p.D, d, row[Nq + Nk + w]);
    }
}

struct DmLayout {
    size_t qkv, Qbuf, Obuf, attn_len, ones, o_rows, last_rows, mask, o, h1, gu, total;
};

DmLayout dm_layout(const ctcsd_config& c, int R, int I) {
    DmLayout l;
    const size_t esz = c.dtype == CTCSD_DTYPE_BF16 ? 2 : 4;
    const size_t W = (c.max_nodes + 63) / 64;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = align_up(off + bytes, 256); return at; };
    l.qkv = take((size_t)c.B * R * (c.Hq + 2 * c.Hkv) * c.D * 4);
    l.Qbuf = take((size_t)c.B * c.max_nodes * c.Hq * c.D * esz);
    l.Obuf = take((size_t)c.B * c.max_nodes * c.Hq * c.D * esz);
    l.attn_len = take((size_t)c.B * 4);
    l.ones = take((size_t)c.B * 4);
    l.o_rows = take((size_t)c.B * 4);
    l.last_rows = take((size_t)c.B * 4);
    l.mask = take((size_t)c.B * c.max_nodes * W * 8);
    l.o = take((size_t)c.B * c.H * 4);
    l.h1 = take((size_t)c.B * c.H * 4);
    l.gu = take((size_t)c.B * 2 * I * 4);
    l.total = off;
    return l;
}

// y[M,N] = x[rows picked by x_rows][K] . W[N,K]^T as float32, through the weight-streaming kernel.
// `act` is applied to the rows of x on the way in; add / y_t: see GemvParams::plain_add, plain_out_t.
int plain_gemv(Handle* h, cudaStream_t s, int M, const void* x, int x_row_count, const int* x_rows, const void* W,
               int K, int N, float* y, const ActOp& act, const float* add = nullptr, void* y_t = nullptr) {
    GemvParams g;
    memset(&g, 0, sizeof(g));
    g.x = x; g.x_rows = x_rows; g.x_row_count = x_row_count; g.W = W;
    g.H = K; g.slots = 1; g.rows_per_slot = N;
    g.mode = 2; g.k = 1;
    g.logits_dbg = y;
    g.act = act; g.plain_add = add; g.plain_out_t = y_t;
    g.sn.max_nodes = 1; g.sn.rows_per_seq = 1; g.sn.inv_temp = 1.f;
    return launch_gemv_stream(h, s, h->cfg.dtype, M, g);
}

template <typename T>
int run_draft_module(Handle* h, cudaStream_t s, DmParams& p, const void* Wqkv, const void* Wo, const void* Wgu,
                     const void* Wdn) {
    const ctcsd_config& c = h->cfg;
    const int Nqkv = (c.Hq + 2 * c.Hkv) * c.D;
    ActOp none = {};
    // q, k, v of every new row: RMSNorm(F) * g1 on the way in (rows past n_new[b] count as zero)
    ActOp norm1 = {};
    norm1.op = 1; norm1.eps = p.eps; norm1.gain = p.g1; norm1.n_new = p.n_new; norm1.R = p.R;
    int rc = plain_gemv(h, s, p.B * p.R, p.F_new, p.B * p.R, nullptr, Wqkv, c.H, Nqkv, p.qkv, norm1);
    if (rc != CTCSD_OK) return rc;
    CTCSD_CUDA_CHECK(h, launch_pdl(dm_rope_scatter_kernel<T>, dim3(p.R, p.B, 8), dim3(256), 0, s, 1, p));
    CTCSD_LAUNCH_CHECK(h);
    AttnParams ap;
    ap.Q = p.Qbuf; ap.K = p.Kd; ap.V = p.Vd; ap.O = p.Obuf;
    ap.kv_len = p.attn_len; ap.n_nodes = p.ones; ap.mask = p.mask;
    ap.B = c.B; ap.Hq = c.Hq; ap.Hkv = c.Hkv; ap.D = c.D; ap.max_nodes = c.max_nodes; ap.Lcap = p.Lcap;
    ap.scale = 1.0f / sqrtf((float)c.D);
    ap.status = p.status;
    rc = tree_attention_dispatch(h, s, ap);
    if (rc != CTCSD_OK) return rc;
    rc = plain_gemv(h, s, p.B, p.Obuf, p.B * c.max_nodes, p.o_rows, Wo, c.Hq * c.D, c.H, p.o, none);
    if (rc != CTCSD_OK) return rc;
    // gate and up: h1 = F_last + o (kept for the last residual), RMSNorm(h1) * g2 on the way in
    ActOp norm2 = {};
    norm2.op = 2; norm2.eps = p.eps; norm2.gain = p.g2; norm2.add = p.o; norm2.sum_out = p.h1;
    rc = plain_gemv(h, s, p.B, p.F_new, p.B * p.R, p.last_rows, Wgu, c.H, 2 * p.I, p.gu, norm2);
    if (rc != CTCSD_OK) return rc;
    // down: SiLU(gate) * up on the way in, F_hat = h1 + product on the way out
    ActOp swiglu = {};
    swiglu.op = 3; swiglu.gu = p.gu;
    rc = plain_gemv(h, s, p.B, p.gu, p.B, nullptr, Wdn, p.I, c.H, p.out_F_dbg, swiglu, p.h1, p.out_F);
    return rc;
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
    for (int i = 0; i < c.D / 2; ++i) p.inv_freq[i] = exp2(-2.0 * (double)i / (double)c.D * log2((double)layer->rope_theta));
    p.qkv = reinterpret_cast<float*>(ws + l.qkv);
    p.Qbuf = ws + l.Qbuf; p.Obuf = ws + l.Obuf;
    p.attn_len = reinterpret_cast<int*>(ws + l.attn_len); p.ones = reinterpret_cast<int*>(ws + l.ones);
    p.o_rows = reinterpret_cast<int*>(ws + l.o_rows); p.last_rows = reinterpret_cast<int*>(ws + l.last_rows);
    p.mask = reinterpret_cast<unsigned long long*>(ws + l.mask);
    p.o = reinterpret_cast<float*>(ws + l.o); p.h1 = reinterpret_cast<float*>(ws + l.h1);
    p.gu = reinterpret_cast<float*>(ws + l.gu);
    p.out_F = out_F; p.out_F_dbg = out_F_dbg; p.out_kv_len = out_kv_len;
    p.status = status_ptr(h);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (c.dtype == CTCSD_DTYPE_BF16)
        return run_draft_module<__nv_bfloat16>(h, s, p, layer->Wqkv, layer->Wo, layer->Wgu, layer->Wdn);
    return run_draft_module<float>(h, s, p, layer->Wqkv, layer->Wo, layer->Wgu, layer->Wdn);
}
