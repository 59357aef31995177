// Tree attention for bf16 on tensor cores: a flash-style kernel that streams the KV cache
// once per (sequence, kv head), split along the KV axis, plus a small merge kernel.
//
// Work decomposition: CTA = (64 query rows, one KV split, kv head g, sequence b).  Query row
// r of kv head g is (node i = r / grp, query head g*grp + r % grp), so all query heads that
// share a kv head read its keys and values from the same shared-memory tile (GQA grouping).
// Each of the 4 warps owns 16 rows: S = Q K^T with mma.m16n8k16 (bf16 in, fp32 out), the
// ancestor mask is applied to the columns that are tree nodes, an online softmax keeps the
// running max and sum, and O += P V reuses the S accumulators as the A operand.  K and V
// tiles of 64 keys are double buffered with cp.async into XOR-swizzled shared memory.
// Every CTA writes (max, sum, unnormalised O) per row; the merge kernel combines the splits.
#include "tree_attention.cuh"

#include <math.h>
#include <string.h>

namespace ctcsd {
namespace {

constexpr int kRows = 64;          // query rows per CTA
constexpr int kKeys = 64;          // keys per tile
constexpr int kThreads = 128;
constexpr int kStages = 4;         // K/V tile buffers: three tiles are in flight while one is used

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool valid) {
    const int bytes = valid ? 16 : 0;                 // 0 source bytes -> the 16 bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// ---- thread-block cluster helpers (distributed shared memory) ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of the same shared-memory location in the CTA with rank `rank` of this cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float2 ld_cluster_v2(uint32_t addr) {
    float2 v;
    asm volatile("ld.shared::cluster.v2.f32 {%0,%1}, [%2];" : "=f"(v.x), "=f"(v.y) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ float4 ld_cluster_v4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}

// byte offset of 16-byte chunk `chunk` of row `row` in a tile with D bf16 per row, swizzled
template <int D> __device__ __forceinline__ uint32_t tile_off(int row, int chunk) {
    return (uint32_t)(row * (D * 2) + ((chunk ^ (row & 7)) << 4));
}

// CLUSTER = false: every CTA writes its partial (max, sum, unnormalised O) rows to `part` and a
// second kernel merges the KV splits.  CLUSTER = true: the `splits` CTAs of a query tile form a
// thread-block cluster, leave their partial rows in their own shared memory, and every CTA
// merges a share of the rows by reading its peers' shared memory; `part` is not used.  In this
// mode the CTA has two groups of four warps: each group takes half of the keys of every tile
// and keeps its own running softmax state, which shortens the dependent instruction chain per
// tile; the two states are simply two more partials for the merge.
template <int D, bool CLUSTER>
__global__ void __launch_bounds__(kThreads * (CLUSTER ? 2 : 1)) tree_attention_mma_kernel(AttnParams p, float* part, int splits) {
    constexpr int KG = CLUSTER ? 2 : 1;        // key groups (warps 4*kg .. 4*kg+3)
    constexpr int NT = kThreads * KG;          // threads per CTA
    constexpr int KPW = kKeys / KG;            // keys of a tile handled by one warp
    constexpr int CH = D / 8;                  // 16-byte chunks per row
    constexpr int KS = D / 16;                 // k-steps of the QK^T product
    constexpr int DT = D / 8;                  // 8-wide output tiles of O
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* Qs = smem;                                  // [64][D]
    unsigned char* Ks = Qs + kRows * D * 2;                    // [kStages][64][D]
    unsigned char* Vs = Ks + kStages * kKeys * D * 2;          // [kStages][64][D]

    const int grp = p.Hq / p.Hkv;
    const int qtile = blockIdx.x / splits, split = blockIdx.x - qtile * splits;
    const int g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, wfull = tid >> 5, lane = tid & 31;
    const int warp = wfull & 3, kg = wfull >> 2;               // row group, key group
    const int gid = lane >> 2, tig = lane & 3;

    pdl_wait();                      // the tree (node count, mask) comes from the preceding kernel
    pdl_trigger();
    int n = p.n_nodes[b];
    int L = p.kv_len[b];
    if (n < 0 || n > p.max_nodes || L < 0 || L + n > p.Lcap) {
        // a sequence that would read outside the cache is treated as empty: no key is loaded
        if (tid == 0) report_error(p.status, CTCSD_ERR_INVALID_ARG, b);
        n = 0;
        L = 0;
    }
    const int Ltot = L + n;
    const int nblk = (Ltot + kKeys - 1) / kKeys;
    const int blk0 = (int)((long long)nblk * split / splits);           // key blocks spread evenly over the splits
    const int blk1 = (int)((long long)nblk * (split + 1) / splits);

    const __nv_bfloat16* Qg = reinterpret_cast<const __nv_bfloat16*>(p.Q);
    const __nv_bfloat16* Kg = reinterpret_cast<const __nv_bfloat16*>(p.K) + ((size_t)b * p.Hkv + g) * (size_t)p.Lcap * D;
    const __nv_bfloat16* Vg = reinterpret_cast<const __nv_bfloat16*>(p.V) + ((size_t)b * p.Hkv + g) * (size_t)p.Lcap * D;

    // rows of this thread: r0 = first row of the pair (gid), r1 = r0 + 8
    const int row_base = qtile * kRows + warp * 16;
    const int rA = row_base + gid, rB = rA + 8;
    const int iA = rA / grp, iB = rB / grp;                     // tree node of each row
    const bool liveA = iA < n, liveB = iB < n;
    const bool warp_live = row_base / grp < n;                  // rows ascend: if the first is dead, all 16 are
    const int W = (p.max_nodes + 63) / 64;
    unsigned long long mA0 = 0, mA1 = 0, mB0 = 0, mB1 = 0;
    if (liveA) { const unsigned long long* m = p.mask + ((size_t)b * p.max_nodes + iA) * W; mA0 = m[0]; if (W > 1) mA1 = m[1]; }
    if (liveB) { const unsigned long long* m = p.mask + ((size_t)b * p.max_nodes + iB) * W; mB0 = m[0]; if (W > 1) mB1 = m[1]; }

    auto load_kv = [&](int blk, int buf) {
        const int key0 = blk * kKeys;
        unsigned char* kd = Ks + buf * (kKeys * D * 2);
        unsigned char* vd = Vs + buf * (kKeys * D * 2);
        for (int c = tid; c < kKeys * CH; c += NT) {
            const int row = c / CH, ch = c - row * CH;
            const int key = key0 + row;
            const bool ok = key < Ltot;
            const size_t src = (size_t)(ok ? key : 0) * D + ch * 8;
            cp_async16(kd + tile_off<D>(row, ch), Kg + src, ok);
            cp_async16(vd + tile_off<D>(row, ch), Vg + src, ok);
        }
    };

    // Q tile (rows past the live rows are zero-filled) and the first KV tile
    for (int c = tid; c < kRows * CH; c += NT) {
        const int row = c / CH, ch = c - row * CH;
        const int r = qtile * kRows + row;
        const int i = r / grp, hq = g * grp + (r - i * grp);
        const bool ok = i < n;
        const size_t src = (((size_t)b * p.max_nodes + (ok ? i : 0)) * p.Hq + hq) * D + ch * 8;
        cp_async16(Qs + tile_off<D>(row, ch), Qg + src, ok);
    }
    // one commit group per tile (possibly empty), so that "all but the newest kStages-1 groups
    // are complete" always means "the tile about to be used has landed"
#pragma unroll
    for (int pre = 0; pre < kStages - 1; ++pre) {
        if (blk0 + pre < blk1) load_kv(blk0 + pre, pre);
        cp_async_commit();
    }

    float o[DT][4];
#pragma unroll
    for (int t = 0; t < DT; ++t) { o[t][0] = o[t][1] = o[t][2] = o[t][3] = 0.f; }
    float mxA = -INFINITY, mxB = -INFINITY, sumA = 0.f, sumB = 0.f;
    const float sl2 = p.scale * 1.4426950408889634f;          // scores are kept in log2 units
    uint32_t qf[KS][4];

    for (int blk = blk0; blk < blk1; ++blk) {
        const int buf = (blk - blk0) % kStages;
        if (blk + kStages - 1 < blk1) load_kv(blk + kStages - 1, (blk - blk0 + kStages - 1) % kStages);
        cp_async_commit();
        cp_async_wait<kStages - 1>();
        __syncthreads();
        if (blk == blk0) {
#pragma unroll
            for (int kk = 0; kk < KS; ++kk) {
                const int row = warp * 16 + (lane & 15), ch = 2 * kk + (lane >> 4);
                ldmatrix_x4(qf[kk], smem_u32(Qs + tile_off<D>(row, ch)));
            }
        }
        const unsigned char* kb = Ks + buf * (kKeys * D * 2);
        const unsigned char* vb = Vs + buf * (kKeys * D * 2);
        if (warp_live) {                                        // warps whose 16 rows are all beyond the tree skip the math

        // S = Q K^T for 16 rows x this warp's KPW keys of the tile.  The k-steps feed NCH separate
        // accumulator sets that are added afterwards: a tensor-core instruction has a long
        // latency, and one accumulator per tile would chain all D/16 of them.
        constexpr int NCH = CLUSTER ? 4 : 2;
        float sp[NCH][KPW / 8][4];
#pragma unroll
        for (int c = 0; c < NCH; ++c)
#pragma unroll
            for (int t = 0; t < KPW / 8; ++t) { sp[c][t][0] = sp[c][t][1] = sp[c][t][2] = sp[c][t][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < KS; ++kk) {
#pragma unroll
            for (int pr = 0; pr < KPW / 16; ++pr) {
                uint32_t kf[4];
                const int mi = lane >> 3, rin = lane & 7;
                const int key = kg * KPW + 16 * pr + (mi >> 1) * 8 + rin, ch = 2 * kk + (mi & 1);
                ldmatrix_x4(kf, smem_u32(kb + tile_off<D>(key, ch)));
                mma_bf16(sp[kk % NCH][2 * pr], qf[kk], kf[0], kf[1]);
                mma_bf16(sp[kk % NCH][2 * pr + 1], qf[kk], kf[2], kf[3]);
            }
        }
        float s[KPW / 8][4];
#pragma unroll
        for (int t = 0; t < KPW / 8; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float v = sp[0][t][e];
#pragma unroll
                for (int c = 1; c < NCH; ++c) v += sp[c][t][e];
                s[t][e] = v;
            }

        // scale, mask, online softmax
        const int key0 = blk * kKeys;
        const bool need_mask = key0 + kKeys > L;
        float bmA = -INFINITY, bmB = -INFINITY;
#pragma unroll
        for (int t = 0; t < KPW / 8; ++t) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float v = s[t][e] * sl2;
                const bool second = e >= 2;                     // c2,c3 belong to row gid+8
                bool vis = second ? liveB : liveA;
                if (need_mask) {
                    const int key = key0 + kg * KPW + 8 * t + 2 * tig + (e & 1);
                    if (key >= L) {
                        const int tn = key - L;
                        const unsigned long long w0 = second ? mB0 : mA0, w1 = second ? mB1 : mA1;
                        unsigned long long w = tn < 64 ? w0 : w1;
                        if (tn >= 128)                          // words past the two kept in registers
                            w = (vis && key < Ltot) ? p.mask[((size_t)b * p.max_nodes + (second ? iB : iA)) * W + (tn >> 6)] : 0ull;
                        vis = vis && key < Ltot && ((w >> (tn & 63)) & 1ull);
                    }
                }
                v = vis ? v : -INFINITY;
                s[t][e] = v;
                if (second) bmB = fmaxf(bmB, v); else bmA = fmaxf(bmA, v);
            }
        }
        bmA = fmaxf(bmA, __shfl_xor_sync(0xffffffffu, bmA, 1));
        bmA = fmaxf(bmA, __shfl_xor_sync(0xffffffffu, bmA, 2));
        bmB = fmaxf(bmB, __shfl_xor_sync(0xffffffffu, bmB, 1));
        bmB = fmaxf(bmB, __shfl_xor_sync(0xffffffffu, bmB, 2));
        const float nmA = fmaxf(mxA, bmA), nmB = fmaxf(mxB, bmB);
        const float refA = nmA == -INFINITY ? 0.f : nmA, refB = nmB == -INFINITY ? 0.f : nmB;
        const float corrA = exp2f(mxA - refA), corrB = exp2f(mxB - refB);   // exp2(-inf) = 0
        mxA = nmA; mxB = nmB;
        float psA = 0.f, psB = 0.f;
        uint32_t pf[KPW / 16][4];
#pragma unroll
        for (int t = 0; t < KPW / 8; ++t) {
            const float p0 = exp2f(s[t][0] - refA), p1 = exp2f(s[t][1] - refA);
            const float p2 = exp2f(s[t][2] - refB), p3 = exp2f(s[t][3] - refB);
            psA += p0 + p1;
            psB += p2 + p3;
            pf[t >> 1][(t & 1) * 2 + 0] = pack_bf16(p0, p1);
            pf[t >> 1][(t & 1) * 2 + 1] = pack_bf16(p2, p3);
        }
        sumA = sumA * corrA + psA;
        sumB = sumB * corrB + psB;
#pragma unroll
        for (int t = 0; t < DT; ++t) { o[t][0] *= corrA; o[t][1] *= corrA; o[t][2] *= corrB; o[t][3] *= corrB; }

        // O += P V
#pragma unroll
        for (int kk = 0; kk < KPW / 16; ++kk) {
#pragma unroll
            for (int pr = 0; pr < DT / 2; ++pr) {
                uint32_t vf[4];
                const int mi = lane >> 3, rin = lane & 7;
                const int key = kg * KPW + 16 * kk + (mi & 1) * 8 + rin, ch = 2 * pr + (mi >> 1);
                ldmatrix_x4_trans(vf, smem_u32(vb + tile_off<D>(key, ch)));
                mma_bf16(o[2 * pr], pf[kk], vf[0], vf[1]);
                mma_bf16(o[2 * pr + 1], pf[kk], vf[2], vf[3]);
            }
        }
        }
        __syncthreads();                                        // the other buffer may be overwritten next
    }
    cp_async_wait<0>();

    sumA += __shfl_xor_sync(0xffffffffu, sumA, 1);
    sumA += __shfl_xor_sync(0xffffffffu, sumA, 2);
    sumB += __shfl_xor_sync(0xffffffffu, sumB, 1);
    sumB += __shfl_xor_sync(0xffffffffu, sumB, 2);
    if constexpr (!CLUSTER) {
        // per-row partials: [b][hq][node][split][D+2] = (max in log2 units, sum, unnormalised O)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = half ? rB : rA;
            const int i = half ? iB : iA;
            if (i >= n) continue;                                   // dead rows are zeroed by the merge kernel
            const int hq = g * grp + (r - i * grp);
            float* dst = part + ((((size_t)b * p.Hq + hq) * p.max_nodes + i) * splits + split) * (D + 2);
            if (tig == 0) { dst[0] = half ? mxB : mxA; dst[1] = half ? sumB : sumA; }
#pragma unroll
            for (int t = 0; t < DT; ++t) {
                float2 v = half ? make_float2(o[t][2], o[t][3]) : make_float2(o[t][0], o[t][1]);
                *reinterpret_cast<float2*>(dst + 2 + 8 * t + 2 * tig) = v;
            }
        }
    } else {
        // partial rows go to this CTA's shared memory (the K/V tiles are no longer needed):
        // [row][D+4] floats = unnormalised O, then max (log2 units) and sum.  Key group 1 writes
        // first; key group 0 folds those values into its own registers and writes the result.
        constexpr int RS = D + 4;
        constexpr int PER = D / 32;
        __syncthreads();
        float* rowbuf = reinterpret_cast<float*>(Ks);
        if (kg == 1) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float* dst = rowbuf + (warp * 16 + gid + 8 * half) * RS;
                if (tig == 0) { dst[D] = half ? mxB : mxA; dst[D + 1] = half ? sumB : sumA; }
#pragma unroll
                for (int t = 0; t < DT; ++t) {
                    float2 v = half ? make_float2(o[t][2], o[t][3]) : make_float2(o[t][0], o[t][1]);
                    *reinterpret_cast<float2*>(dst + 8 * t + 2 * tig) = v;
                }
            }
        }
        __syncthreads();
        if (kg == 0) {
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                float* dst = rowbuf + (warp * 16 + gid + 8 * half) * RS;
                const float m0 = half ? mxB : mxA, l0 = half ? sumB : sumA;
                const float m1 = dst[D], l1 = dst[D + 1];
                const float gm = fmaxf(m0, m1);
                const float w0 = (m0 == -INFINITY) ? 0.f : exp2f(m0 - gm);
                const float w1 = (m1 == -INFINITY) ? 0.f : exp2f(m1 - gm);
                __syncwarp();                                       // every lane of the quad has read max and sum
                if (tig == 0) { dst[D] = gm; dst[D + 1] = w0 * l0 + w1 * l1; }
#pragma unroll
                for (int t = 0; t < DT; ++t) {
                    float2* q = reinterpret_cast<float2*>(dst + 8 * t + 2 * tig);
                    const float2 v1 = *q;
                    const float2 v0 = half ? make_float2(o[t][2], o[t][3]) : make_float2(o[t][0], o[t][1]);
                    *q = make_float2(w0 * v0.x + w1 * v1.x, w0 * v0.y + w1 * v1.y);
                }
            }
        }
        cluster_sync_all();
        // this CTA (cluster rank = split) merges rows split, split + splits, ...; one warp per row
        const uint32_t base = smem_u32(rowbuf);
        for (int rl = split + splits * wfull; rl < kRows; rl += splits * (NT / 32)) {
            const int r = qtile * kRows + rl;
            const int i = r / grp;
            if (i >= p.max_nodes) continue;                         // padding rows of the last query tile
            const int hq = g * grp + (r - i * grp);
            __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.O) + (((size_t)b * p.max_nodes + i) * p.Hq + hq) * D;
            float acc[PER], tot = 0.f;
#pragma unroll
            for (int d = 0; d < PER; ++d) acc[d] = 0.f;
            if (i < n) {                                            // uniform over the warp
                // lane c fetches split c's (max, sum); the row loads below do not depend on one another
                float m_l = -INFINITY, l_l = 0.f;
                if (lane < splits) {
                    const uint32_t a = map_to_cta(base + (uint32_t)(rl * RS + D) * 4u, (uint32_t)lane);
                    const float2 ml = ld_cluster_v2(a);
                    m_l = ml.x;
                    l_l = ml.y;
                }
                const float gm = warp_max(m_l);
                const float w_l = (m_l == -INFINITY) ? 0.f : exp2f(m_l - gm);
                tot = warp_sum(w_l * l_l);
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    if (c < splits) {
                        const float w = __shfl_sync(0xffffffffu, w_l, c);
                        const uint32_t rowaddr = map_to_cta(base + (uint32_t)(rl * RS) * 4u, (uint32_t)c);
                        if constexpr (PER == 4) {
                            const float4 v = ld_cluster_v4(rowaddr + (uint32_t)lane * 16u);
                            acc[0] += w * v.x; acc[1] += w * v.y; acc[2] += w * v.z; acc[3] += w * v.w;
                        } else {
                            const float2 v = ld_cluster_v2(rowaddr + (uint32_t)lane * 8u);
                            acc[0] += w * v.x; acc[1] += w * v.y;
                        }
                    }
                }
            }
            const float inv = tot > 0.f ? 1.f / tot : 0.f;
            if constexpr (PER == 4) {
                uint2 pk;
                pk.x = pack_bf16(acc[0] * inv, acc[1] * inv);
                pk.y = pack_bf16(acc[2] * inv, acc[3] * inv);
                *reinterpret_cast<uint2*>(out + 4 * lane) = pk;
            } else {
                *reinterpret_cast<uint32_t*>(out + 2 * lane) = pack_bf16(acc[0] * inv, acc[1] * inv);
            }
        }
        // nobody may leave while a peer can still read its shared memory
        cluster_sync_all();
    }
}

// One warp per (sequence, node, query head): combine the KV splits and write bf16.
template <int D>
__global__ void __launch_bounds__(128) tree_attention_merge_kernel(AttnParams p, const float* part, int splits) {
    const int lane = threadIdx.x & 31;
    const long long wid = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
    const long long total = (long long)p.B * p.max_nodes * p.Hq;
    if (wid >= total) return;
    const int hq = (int)(wid % p.Hq);
    const int i = (int)((wid / p.Hq) % p.max_nodes);
    const int b = (int)(wid / ((long long)p.Hq * p.max_nodes));
    const float* src = part + (((size_t)b * p.Hq + hq) * p.max_nodes + i) * splits * (D + 2);
    int n = p.n_nodes[b];
    const int L = p.kv_len[b];
    if (n < 0 || n > p.max_nodes || L < 0 || L + n > p.Lcap) n = 0;
    float gm = -INFINITY;
    if (i < n)
        for (int s = 0; s < splits; ++s) gm = fmaxf(gm, src[(size_t)s * (D + 2)]);
    constexpr int PER = D / 32;
    float acc[PER], tot = 0.f;
#pragma unroll
    for (int d = 0; d < PER; ++d) acc[d] = 0.f;
    if (gm != -INFINITY) {
        for (int s = 0; s < splits; ++s) {
            const float* ps = src + (size_t)s * (D + 2);
            const float m = ps[0];
            if (m == -INFINITY) continue;
            const float w = exp2f(m - gm);
            tot += w * ps[1];
#pragma unroll
            for (int d = 0; d < PER; ++d) acc[d] += w * ps[2 + lane + 32 * d];
        }
    }
    const float inv = tot > 0.f ? 1.f / tot : 0.f;
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.O) + (((size_t)b * p.max_nodes + i) * p.Hq + hq) * D;
#pragma unroll
    for (int d = 0; d < PER; ++d) out[lane + 32 * d] = __float2bfloat16_rn(acc[d] * inv);
}

// The KV splits of a query tile run as one thread-block cluster and merge through distributed
// shared memory: one launch, no partial results in global memory.
template <int D>
int launch_d(Handle* h, cudaStream_t s, const AttnParams& p) {
    const int grp = p.Hq / p.Hkv;
    const int qtiles = (p.max_nodes * grp + kRows - 1) / kRows;
    // as many KV splits as still run in one wave (one CTA per SM), as a cluster size that is
    // portable: 1, 2, 4 or 8
    const long long units = (long long)p.B * p.Hkv * qtiles;
    int splits = 1;
    while (splits < 8 && units * splits * 2 <= (long long)h->num_sms) splits *= 2;
    const size_t smem = (size_t)kRows * D * 2 + 2 * kStages * (size_t)kKeys * D * 2;
    auto kern = tree_attention_mma_kernel<D, true>;
    CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    float* no_part = nullptr;
    CTCSD_CUDA_CHECK(h, launch_pdl(kern, dim3(qtiles * splits, p.Hkv, p.B), dim3(kThreads * 2), smem, s, splits,
                                   p, no_part, splits));
    h->launches++;
    return CTCSD_OK;
}

// Same two launches with the partial buffer and the split count given by the caller of this
// function instead of a handle's workspace.  `part` holds B*Hq*max_nodes*splits*(D+2) floats.
template <int D>
cudaError_t launch_d_scratch(cudaStream_t s, const AttnParams& p, float* part, int splits) {
    const int grp = p.Hq / p.Hkv;
    const int qtiles = (p.max_nodes * grp + kRows - 1) / kRows;
    const size_t smem = (size_t)kRows * D * 2 + 2 * kStages * (size_t)kKeys * D * 2;
    auto kern = tree_attention_mma_kernel<D, false>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    dim3 grid(qtiles * splits, p.Hkv, p.B);
    kern<<<grid, kThreads, smem, s>>>(p, part, splits);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const long long warps = (long long)p.B * p.max_nodes * p.Hq;
    tree_attention_merge_kernel<D><<<(unsigned)((warps + 3) / 4), 128, 0, s>>>(p, part, splits);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_tree_attention_mma_scratch(cudaStream_t s, const AttnParams& p, float* part, int splits) {
    if (p.D == 64) return launch_d_scratch<64>(s, p, part, splits);
    return launch_d_scratch<128>(s, p, part, splits);
}

int launch_tree_attention_mma(Handle* h, cudaStream_t s, const AttnParams& p) {
    if (p.D == 64) return launch_d<64>(h, s, p);
    return launch_d<128>(h, s, p);
}

}  // namespace ctcsd
