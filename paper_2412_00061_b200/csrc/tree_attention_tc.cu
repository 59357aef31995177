// Tree attention for bf16 on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// Work decomposition: CTA = (128 query rows, one KV split, kv head g, sequence b).  Query row
// r of kv head g is (node i = r / grp, query head g*grp + r % grp), so all query heads that
// share a kv head use the same K/V tiles (GQA grouping).  Per tile of 128 keys:
//   S[128 x 128] = Q K^T        tcgen05.mma, both operands K-major from shared memory (TMA,
//                               128-byte swizzle), accumulator in tensor memory;
//   softmax                     eight warps, two threads per query row: the row is read from
//                               tensor memory twice (max, then exp2 and sum), the ancestor mask
//                               is applied to the columns that are tree nodes, P goes to shared
//                               memory as bf16 in the K-major swizzled layout;
//   O_tile[128 x D] = P V       tcgen05.mma with V as an MN-major operand (V is [key][d]);
//   O = O * corr + O_tile       in the row's registers.
// Warp 0 issues the TMA loads (Q once, K/V tiles into a two-stage ring), warp 1 issues the
// MMAs, warps 2..9 are the softmax warps (two threads per query row: each takes half of a tile's keys
// and half of O's columns).  The KV splits of a query tile form a thread-block
// cluster and merge their (max, sum, O) rows through distributed shared memory.
#include "tree_attention.cuh"
#include "tc_primitives.cuh"

#include <math.h>
#include <string.h>

namespace ctcsd {
namespace {

constexpr int kSoftmaxWarps = 8;     // two per quarter of the TMEM lanes
constexpr int kThreads = 64 + 32 * kSoftmaxWarps;
constexpr int kRows = 128;         // query rows per CTA
constexpr int kKeys = 128;         // keys per tile
constexpr int kStages = 3;         // K/V tile buffers: the tile in use, and two on their way
constexpr float kSlack = 8.f;      // how far (log2 units) the row maximum may run ahead of the exponent's reference

struct __align__(8) AttnShared {
    uint64_t q_full;
    uint64_t full[kStages];        // K and V tile landed
    uint64_t empty[kStages];       // both MMAs of the tile have read it
    uint64_t s_full[2];            // S of an even / odd tile is in tensor memory
    uint64_t p_full[2];            // P of an even / odd tile is in shared memory (and S has been read).  Two
                                   // barriers: a softmax warp may finish tile t+1 while another still writes P
                                   // of tile t (it cannot reach tile t+2, whose S is issued after P of t is complete),
                                   // and its arrival must not count for tile t
    uint64_t o_full;               // O_tile is in tensor memory
    uint32_t tmem_base;
    int abort_flag;
    int never_set;
    float xch[2][2][kRows];        // row maxima (two tile parities; the row sums at the end take the free parity) exchanged between a row's two threads
};

// The two softmax warps that share a quarter of the TMEM lanes (64 threads) meet here.
__device__ __forceinline__ void pair_barrier(int q) {
    asm volatile("bar.sync %0, 64;" ::"r"(q + 1) : "memory");
}

__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
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
// 2^x for x <= 0 (the softmax exponent is never positive): the hardware approximation, no range fix-up
__device__ __forceinline__ float exp2_fast(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
tree_attention_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                         const __grid_constant__ CUtensorMap tmV, AttnParams p, int splits) {
    constexpr int DH = D / 64;                     // 64-column halves of a row of D elements
    constexpr int kQBytes = kRows * D * 2;
    constexpr int kTileBytes = kKeys * D * 2;      // one K or V tile
    constexpr int kPBytes = kRows * kKeys * 2;
    constexpr int RS = D + 4;                      // floats per row of the merge buffer
    constexpr int PER = D / 32;
    constexpr int DO = D / 2;                      // O columns per softmax thread
    // The tiles need 1024-byte alignment (128-byte swizzle); with three 64 KB stages there is no room
    // left for an alignment pad, so the alignment is asked for and checked.
    extern __shared__ __align__(1024) unsigned char dyn[];
    unsigned char* Qs = dyn;                                           // [DH][128 rows][128 B]
    unsigned char* KV = Qs + kQBytes;                                  // [kStages][K tile | V tile]
    // P (128 rows x 128 keys of bf16 = 32 KB) has the shape of a K tile with D = 128, and by the time
    // it is written the tile's K has served its purpose (S is complete): P takes K's place in the
    // stage.  With D = 64 a K tile is half that size and P has a buffer of its own.
    constexpr bool kPInK = (kTileBytes >= kPBytes);
    unsigned char* Ps_own = KV + kStages * 2 * kTileBytes;             // [2][128 rows][128 B], D = 64 only
    AttnShared* sh = reinterpret_cast<AttnShared*>(Ps_own + (kPInK ? 0 : kPBytes));
    auto p_tile = [&](int s) -> unsigned char* { return kPInK ? KV + (size_t)s * 2 * kTileBytes : Ps_own; };
    if ((tc::smem_u32(dyn) & 1023u) != 0u) {                           // uniform over the CTA (and its cluster)
        if (threadIdx.x == 0) report_error(p.status, CTCSD_ERR_INTERNAL, 24);
        return;
    }

    const int grp = p.Hq / p.Hkv;
    const int qtile = blockIdx.x / splits, split = blockIdx.x - qtile * splits;
    const int g = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort_flag = &sh->abort_flag;

    if (tid == 0) {
        tc::mbar_init(&sh->q_full, 1);
        for (int s = 0; s < kStages; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], 1); }
        tc::mbar_init(&sh->s_full[0], 1);
        tc::mbar_init(&sh->s_full[1], 1);
        tc::mbar_init(&sh->p_full[0], kSoftmaxWarps);
        tc::mbar_init(&sh->p_full[1], kSoftmaxWarps);
        tc::mbar_init(&sh->o_full, 1);
        sh->abort_flag = 0;
        sh->never_set = 0;
        tc::fence_barrier_init();
    }
    if (warp == 1) {
        tc::tmem_alloc(&sh->tmem_base, 512);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_s = sh->tmem_base;               // S of even tiles: columns 0..127, of odd tiles: 128..255
    const uint32_t tmem_o = sh->tmem_base + 256;         // O_tile: columns 256..256+D-1

    pdl_wait();                      // the tree (node count, mask) and Q/K/V come from preceding kernels
    pdl_trigger();
    int n = p.n_nodes[b];
    int L = p.kv_len[b];
    if (n < 0 || n > p.max_nodes || L < 0 || L + n > p.Lcap) {
        if (tid == 0) report_error(p.status, CTCSD_ERR_INVALID_ARG, b);
        n = 0;
        L = 0;
    }
    const int Ltot = L + n;
    const int nblk = (Ltot + kKeys - 1) / kKeys;
    const int blk0 = (int)((long long)nblk * split / splits);           // key tiles spread evenly over the splits
    const int blk1 = (int)((long long)nblk * (split + 1) / splits);
    // a query tile whose rows all belong to unused nodes has nothing to attend to: its rows come out zero
    const int ntile = (qtile * (kRows / grp) >= n) ? 0 : blk1 - blk0;

    // softmax state of the row owned by this thread (softmax warps only)
    float acc[DO];
    float ref = -INFINITY, sum = 0.f;           // exponent reference (log2 units) and row sum of the softmax
    bool failed = false;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0 && ntile > 0) {
            tc::prefetch_tensormap(&tmQ);
            tc::prefetch_tensormap(&tmK);
            tc::prefetch_tensormap(&tmV);
            const uint64_t pol = tc::policy_evict_last();
            tc::mbar_arrive_expect_tx(&sh->q_full, (uint32_t)kQBytes);
            for (int hh = 0; hh < DH; ++hh)
                tc::tma_load_5d(Qs + hh * (kRows * 128), &tmQ, &sh->q_full, hh * 64, 0, g, qtile * (kRows / grp), b, pol);
            int it = 0;
            for (int blk = blk0; blk < blk1; ++blk, ++it) {
                const int s = it % kStages;
                const uint32_t ph = (uint32_t)(it / kStages) & 1u;
                if (!tc::mbar_wait(&sh->empty[s], ph ^ 1u, abort_flag)) { failed = true; break; }
                unsigned char* kd = KV + (size_t)s * 2 * kTileBytes;
                tc::mbar_arrive_expect_tx(&sh->full[s], (uint32_t)(2 * kTileBytes));
                // one copy per tile and tensor: the box spans both 64-column halves of the head dimension
                // and lands as [half][key][128 bytes] (every copy instruction costs the copy engine a fixed
                // few hundred nanoseconds, whatever its size)
                // one copy per tile and tensor: the box spans all 64-column parts of the head dimension and
                // lands as [part][key][128 bytes] (a copy instruction costs the copy engine a fixed few
                // hundred nanoseconds whatever its size)
                tc::tma_load_5d(kd, &tmK, &sh->full[s], 0, blk * kKeys, 0, g, b, pol);
                tc::tma_load_5d(kd + kTileBytes, &tmV, &sh->full[s], 0, blk * kKeys, 0, g, b, pol);
            }
            if (failed) {
                if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 21);
                *abort_flag = 1;
                for (int back = 1; back <= kStages && back <= it; ++back) {
                    const int j = it - back;
                    tc::mbar_wait(&sh->full[j % kStages], (uint32_t)(j / kStages) & 1u, &sh->never_set, 1ll << 24);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0 && ntile > 0) {
            const uint32_t idesc_s = tc::idesc_bf16_f32(kRows, kKeys);
            const uint32_t idesc_o = tc::idesc_bf16_f32_b_mn(kRows, D);
            bool ok = tc::mbar_wait(&sh->q_full, 0u, abort_flag);
            // S = Q K^T of tile t into S buffer t & 1: D/16 steps of 16 elements along the head dimension.
            // It is issued one tile ahead, so that it runs while the softmax warps work on tile t - 1
            // (they finished reading buffer t & 1 before they released P of tile t - 2).
            auto issue_s = [&](int t) -> bool {
                const int s = t % kStages;
                if (!tc::mbar_wait(&sh->full[s], (uint32_t)(t / kStages) & 1u, abort_flag)) return false;
                tc::tc_fence_after_sync();
                const uint32_t k_addr = tc::smem_u32(KV + (size_t)s * 2 * kTileBytes);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint64_t adesc = tc::smem_desc_k_sw128(tc::smem_u32(Qs) + (kk / 4) * (kRows * 128)) + 2 * (kk % 4);
                    const uint64_t bdesc = tc::smem_desc_k_sw128(k_addr + (kk / 4) * (kKeys * 128)) + 2 * (kk % 4);
                    tc::mma_bf16_ss(tmem_s + (uint32_t)((t & 1) * 128), adesc, bdesc, idesc_s, kk != 0 ? 1u : 0u);
                }
                tc::mma_commit(&sh->s_full[t & 1]);
                return true;
            };
            if (ok) ok = issue_s(0);
            for (int it = 0; it < ntile && ok; ++it) {
                const int s = it % kStages;
                if (it + 1 < ntile && !issue_s(it + 1)) { ok = false; break; }
                const uint32_t v_addr = tc::smem_u32(KV + (size_t)s * 2 * kTileBytes) + kTileBytes;
                // O_tile = P V once the softmax warps have written P (they have then also read S)
                if (!tc::mbar_wait(&sh->p_full[it & 1], (uint32_t)(it >> 1) & 1u, abort_flag)) { ok = false; break; }
                tc::tc_fence_after_sync();
#pragma unroll
                for (int kk = 0; kk < kKeys / 16; ++kk) {
                    const uint64_t adesc = tc::smem_desc_k_sw128(tc::smem_u32(p_tile(s)) + (kk / 4) * (kRows * 128)) + 2 * (kk % 4);
                    // 16 keys further along K = 16 rows of 128 bytes
                    const uint64_t bdesc = tc::smem_desc_mn_sw128(v_addr + kk * (16 * 128), kKeys * 128);
                    tc::mma_bf16_ss(tmem_o, adesc, bdesc, idesc_o, (it | kk) != 0 ? 1u : 0u);   // O accumulates over the tiles
                }
                tc::mma_commit(&sh->o_full);
                tc::mma_commit(&sh->empty[s]);
            }
            if (!ok) {
                if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 22);
                *abort_flag = 1;
            }
        }
    } else {
        // ---------------- softmax warps: two threads per query row ----------------
        // Warps 2..5 take the first 64 keys of a tile and the first D/2 columns of O, warps 6..9
        // the other halves; the two threads of a row meet at a 64-thread named barrier to agree on
        // the tile's maximum.  Every softmax thread executes every one of those barriers, also
        // after a wait has failed, so a failure cannot leave a partner waiting.
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int half = (warp - 2) >> 2;             // which half of the keys / of O's columns
        const int kc0 = half * (kKeys / 2);           // first key column of this thread
        const int oc0 = half * DO;                    // first O column of this thread
        const int rl = q * 32 + lane;                 // row of the tile
        const uint32_t lane_off = (uint32_t)(q * 32) << 16;
        const int r = qtile * kRows + rl;
        const int i = r / grp;                        // tree node of the row
        const bool live = i < n;
        const int W = (p.max_nodes + 63) / 64;
        // the first two mask words live in registers; trees above 128 nodes read the others
        // from memory where a chunk of keys needs them
        unsigned long long m0 = 0, m1 = 0;
        const unsigned long long* mrow = p.mask + ((size_t)b * p.max_nodes + (live ? i : 0)) * W;
        if (live) {
            m0 = mrow[0];
            if (W > 1) m1 = mrow[1];
        }
        auto mask_word = [&](int w) -> unsigned long long {
            return w == 0 ? m0 : (w == 1 ? m1 : (w < W ? mrow[w] : 0ull));
        };
#pragma unroll
        for (int d = 0; d < DO; ++d) acc[d] = 0.f;
        const float sl2 = p.scale * 1.4426950408889634f;          // scores are kept in log2 units
        for (int it = 0; it < ntile; ++it) {
            const int key0 = (blk0 + it) * kKeys;
            const int s = it % kStages;
            if (!failed && !tc::mbar_wait(&sh->s_full[it & 1], (uint32_t)(it >> 1) & 1u, abort_flag)) failed = true;
            failed = __any_sync(0xffffffffu, failed);
            tc::tc_fence_after_sync();
            const bool tail = key0 + kKeys > L;       // the tile holds tree nodes or keys past the end
            // V rows past the last key may hold anything (the cache is only written up to there):
            // clear them, a zero weight does not cancel a NaN
            if (half == 0 && key0 + rl >= Ltot) {
                unsigned char* vrow = KV + (size_t)s * 2 * kTileBytes + kTileBytes + rl * 128;
#pragma unroll
                for (int hh = 0; hh < DH; ++hh)
#pragma unroll
                    for (int c = 0; c < 8; ++c)
                        *reinterpret_cast<uint4*>(vrow + hh * (kKeys * 128) + c * 16) = make_uint4(0, 0, 0, 0);
            }
            // visibility of the 32 keys key0 + c0 .. + 31 for this row as a bit mask: cached keys are
            // visible to every live row, tree node t only if the row's ancestor mask has bit t (bits
            // of nodes past the tree are never set, so keys past the end come out invisible)
            auto visible32 = [&](int c0) -> uint32_t {
                if (!live) return 0u;
                if (!tail) return 0xffffffffu;
                const int t0 = key0 + c0 - L;                   // tree index of the chunk's first key
                if (t0 <= -32) return 0xffffffffu;
                if (t0 < 0) return (uint32_t)((m0 << (-t0)) | ((1ull << (-t0)) - 1ull));
                const int w = t0 >> 6, sft = t0 & 63;
                unsigned long long bits = mask_word(w) >> sft;
                if (sft > 32) bits |= mask_word(w + 1) << (64 - sft);
                return (uint32_t)bits;
            };
            // One pass over the tile in the common case.  P = 2^(S - ref) is formed against the reference
            // the row already has, and the tile's maximum is taken along the way; only when that maximum
            // turns out to lie more than kSlack above the reference (in log2 units; always on the first
            // tile with a visible key) does the reference move: O and the row sum are rescaled and the
            // pass is repeated against the new reference.  P therefore stays below 2^kSlack, and O, which
            // accumulates in tensor memory, rarely needs rescaling.  Both threads of a row see the same
            // numbers and take the same decisions; a warp repeats the pass if any of its rows has to
            // (the tensor-memory loads are warp-wide).
            unsigned char* pt = p_tile(s);
            if (!kPInK) {
                // a single P buffer: the previous tile's P V product must have consumed it
                if (it > 0 && !failed && !tc::mbar_wait(&sh->o_full, (uint32_t)(it - 1) & 1u, abort_flag)) failed = true;
                failed = __any_sync(0xffffffffu, failed);
            }
            float part = 0.f;                              // this thread's share of the tile's row sum
            float bm = -INFINITY;
            auto pass = [&](float rf) {                    // rf: reference in log2 units (finite)
                float ps4[4] = {0.f, 0.f, 0.f, 0.f};
                float bm4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four chains instead of one
#pragma unroll 1
                for (int c0 = kc0; c0 < kc0 + kKeys / 2; c0 += 32) {
                    uint32_t v[32];
                    tc::tmem_ld32(tmem_s + (uint32_t)((it & 1) * 128) + lane_off + (uint32_t)c0, v);
                    const uint32_t vm = visible32(c0);
                    tc::tmem_ld_wait();
                    float pv[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float x = __uint_as_float(v[j]);
                        const bool vis = (vm >> j) & 1u;
                        const float e = exp2_fast(fmaf(x, sl2, -rf));
                        pv[j] = vis ? e : 0.f;
                        ps4[j & 3] += pv[j];
                        bm4[j & 3] = vis ? fmaxf(bm4[j & 3], x) : bm4[j & 3];
                    }
                    unsigned char* prow = pt + (c0 / 64) * (kRows * 128) + rl * 128;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint4 w;
                        w.x = pack_bf16(pv[8 * c + 0], pv[8 * c + 1]);
                        w.y = pack_bf16(pv[8 * c + 2], pv[8 * c + 3]);
                        w.z = pack_bf16(pv[8 * c + 4], pv[8 * c + 5]);
                        w.w = pack_bf16(pv[8 * c + 6], pv[8 * c + 7]);
                        const int chunk = (c0 % 64) / 8 + c;
                        *reinterpret_cast<uint4*>(prow + ((chunk ^ (rl & 7)) << 4)) = w;
                    }
                }
                part = (ps4[0] + ps4[1]) + (ps4[2] + ps4[3]);
                bm = fmaxf(fmaxf(bm4[0], bm4[1]), fmaxf(bm4[2], bm4[3]));
            };
            if (!failed) pass(ref == -INFINITY ? 0.f : ref);
            sh->xch[it & 1][half][rl] = bm;
            pair_barrier(q);
            bm = fmaxf(bm, sh->xch[it & 1][half ^ 1][rl]);
            bm *= sl2;                                 // scale > 0: the maximum commutes with it
            const bool move = bm > ref + kSlack;       // also the first tile with a visible key (ref = -inf)
            if (__any_sync(0xffffffffu, move) && !failed) {
                const float nref = move ? bm : ref;
                const float corr = move ? exp2_fast(ref - nref) : 1.f;     // exp2(-inf) = 0
                // O must be complete before it is rescaled
                if (it > 0) {
                    if (kPInK && !tc::mbar_wait(&sh->o_full, (uint32_t)(it - 1) & 1u, abort_flag)) failed = true;
                    failed = __any_sync(0xffffffffu, failed);
                    if (!failed) {
                        tc::tc_fence_after_sync();
#pragma unroll
                        for (int c0 = 0; c0 < DO; c0 += 32) {
                            uint32_t v[32];
                            tc::tmem_ld32(tmem_o + lane_off + (uint32_t)(oc0 + c0), v);
                            tc::tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * corr);
                            tc::tmem_st32(tmem_o + lane_off + (uint32_t)(oc0 + c0), v);
                        }
                        tc::tmem_st_wait();
                    }
                }
                sum *= corr;
                ref = nref;
                // a row without any visible key so far keeps ref = -inf; its P is all zero whatever the reference
                if (!failed) pass(ref == -INFINITY ? 0.f : ref);
            }
            if (failed) continue;
            sum += part;
            // make P (and the cleared V rows) visible to the tensor core, then hand over
            tc::fence_proxy_async();
            tc::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&sh->p_full[it & 1]);
        }
        // O is complete once the last P V product has landed: fetch this thread's half of the row
        if (ntile > 0 && !failed && !tc::mbar_wait(&sh->o_full, (uint32_t)(ntile - 1) & 1u, abort_flag)) failed = true;
        failed = __any_sync(0xffffffffu, failed);
        if (ntile > 0 && !failed) {
            tc::tc_fence_after_sync();
#pragma unroll
            for (int c0 = 0; c0 < DO; c0 += 32) {
                uint32_t v[32];
                tc::tmem_ld32(tmem_o + lane_off + (uint32_t)(oc0 + c0), v);
                tc::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) acc[c0 + j] = __uint_as_float(v[j]);
            }
            tc::tc_fence_before_sync();
        }
        // the row's sum is the two halves' sums (both were kept against the same running maximum)
        // (the parity the last tile did not use: its previous readers passed a later barrier since)
        sh->xch[ntile & 1][half][rl] = sum;
        pair_barrier(q);
        sum += sh->xch[ntile & 1][half ^ 1][rl];
        if (failed && lane == 0) {
            if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 23);
            *abort_flag = 1;
        }
    }

    // ---------------- output ----------------
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc::tc_fence_after_sync();
        tc::tmem_dealloc(sh->tmem_base, 512);
    }
    const bool good = sh->abort_flag == 0;
    if (splits == 1) {
        if (warp >= 2 && good) {
            const int rl = (warp & 3) * 32 + lane;
            const int half = (warp - 2) >> 2;
            const int r = qtile * kRows + rl;
            const int i = r / grp;
            if (i < p.max_nodes) {
                const int hq = g * grp + (r - i * grp);
                __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.O) +
                                     (((size_t)b * p.max_nodes + i) * p.Hq + hq) * D + half * DO;
                const float inv = (i < n && sum > 0.f) ? 1.f / sum : 0.f;
#pragma unroll
                for (int c = 0; c < DO / 8; ++c) {
                    uint4 w;
                    w.x = pack_bf16(acc[8 * c + 0] * inv, acc[8 * c + 1] * inv);
                    w.y = pack_bf16(acc[8 * c + 2] * inv, acc[8 * c + 3] * inv);
                    w.z = pack_bf16(acc[8 * c + 4] * inv, acc[8 * c + 5] * inv);
                    w.w = pack_bf16(acc[8 * c + 6] * inv, acc[8 * c + 7] * inv);
                    reinterpret_cast<uint4*>(out)[c] = w;
                }
            }
        }
        return;
    }
    // several KV splits: every CTA leaves its rows (unnormalised O, max, sum) in its shared memory
    // (the K/V tiles are no longer needed) and merges rows split, split + splits, ... of all CTAs
    float* rowbuf = reinterpret_cast<float*>(KV);
    if (warp >= 2) {
        const int rl = (warp & 3) * 32 + lane;
        const int half = (warp - 2) >> 2;
        float* dst = rowbuf + rl * RS;
#pragma unroll
        for (int c = 0; c < DO / 4; ++c)
            *reinterpret_cast<float4*>(dst + half * DO + 4 * c) =
                make_float4(acc[4 * c], acc[4 * c + 1], acc[4 * c + 2], acc[4 * c + 3]);
        if (half == 0) {
            dst[D] = ref;                       // the reference the row is expressed against
            dst[D + 1] = sum;                      // already the whole row's sum
        }
    }
    cluster_sync_all();
    const uint32_t base = tc::smem_u32(rowbuf);
    for (int rl = split + splits * warp; rl < kRows && good; rl += splits * (kThreads / 32)) {
        const int r = qtile * kRows + rl;
        const int i = r / grp;
        if (i >= p.max_nodes) continue;                         // padding rows of the last query tile
        const int hq = g * grp + (r - i * grp);
        __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(p.O) + (((size_t)b * p.max_nodes + i) * p.Hq + hq) * D;
        float o[PER], tot = 0.f;
#pragma unroll
        for (int d = 0; d < PER; ++d) o[d] = 0.f;
        if (i < n) {                                            // uniform over the warp
            // lane c fetches split c's (max, sum); the row loads below do not depend on one another
            float m_l = -INFINITY, l_l = 0.f;
            if (lane < splits) {
                const float2 ml = ld_cluster_v2(map_to_cta(base + (uint32_t)(rl * RS + D) * 4u, (uint32_t)lane));
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
                        o[0] += w * v.x; o[1] += w * v.y; o[2] += w * v.z; o[3] += w * v.w;
                    } else {
                        const float2 v = ld_cluster_v2(rowaddr + (uint32_t)lane * 8u);
                        o[0] += w * v.x; o[1] += w * v.y;
                    }
                }
            }
        }
        const float inv = tot > 0.f ? 1.f / tot : 0.f;
        if constexpr (PER == 4) {
            uint2 pk;
            pk.x = pack_bf16(o[0] * inv, o[1] * inv);
            pk.y = pack_bf16(o[2] * inv, o[3] * inv);
            *reinterpret_cast<uint2*>(out + 4 * lane) = pk;
        } else {
            *reinterpret_cast<uint32_t*>(out + 2 * lane) = pack_bf16(o[0] * inv, o[1] * inv);
        }
    }
    // nobody may leave while a peer can still read its shared memory
    cluster_sync_all();
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
    if (qres != cudaDriverEntryPointSuccess) return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(sym);
    return fn;
}

// bf16 tensor of rank `rank`: dims[0] is the contiguous axis, strides[] in bytes for dims 1..;
// box[0] = 64 elements (one 128-byte swizzle row); out-of-range elements read as zero.
bool make_map_nd(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
                 const cuuint32_t* box) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides, box,
                    estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int D>
int launch_tc(Handle* h, cudaStream_t s, const AttnParams& p) {
    const int grp = p.Hq / p.Hkv;
    const int rows_total = p.max_nodes * grp;
    const int qtiles = (rows_total + kRows - 1) / kRows;
    // KV splits as a portable cluster size, all CTAs in one wave (clusters of 8 schedule badly here)
    const long long units = (long long)p.B * p.Hkv * qtiles;
    // (1, 2 or 4: clusters of 8 schedule badly here).  The CTAs run in waves of one per SM; pick
    // the smallest split count whose waves are within 10 % of the shortest total.
    int splits = 1;
    {
        double best = 1e30;
        double cost[3];
        for (int e = 0; e < 3; ++e) {
            const long long ctas = units << e;
            cost[e] = (double)((ctas + h->num_sms - 1) / h->num_sms) / (double)(1 << e) + 0.15 * e;   // a split costs a cluster merge
            if (cost[e] < best) best = cost[e];
        }
        for (int e = 0; e < 3; ++e)
            if (cost[e] <= best * 1.10) { splits = 1 << e; break; }
    }

    CUtensorMap tmQ, tmK, tmV;
    {   // Q [B][max_nodes][Hkv][grp][D]: box = 64 columns x grp heads x 1 kv head x 128/grp nodes x 1 sequence
        cuuint64_t dims[5] = {(cuuint64_t)D, (cuuint64_t)grp, (cuuint64_t)p.Hkv, (cuuint64_t)p.max_nodes, (cuuint64_t)p.B};
        cuuint64_t str[4] = {(cuuint64_t)D * 2, (cuuint64_t)grp * D * 2, (cuuint64_t)p.Hq * D * 2,
                             (cuuint64_t)p.max_nodes * p.Hq * D * 2};
        cuuint32_t box[5] = {64, (cuuint32_t)grp, 1, (cuuint32_t)(kRows / grp), 1};
        if (!make_map_nd(&tmQ, p.Q, 5, dims, str, box)) return CTCSD_ERR_CUDA;
    }
    {   // K, V [B][Hkv][Lcap][D] seen as [B][Hkv][D/64][Lcap][64]: box = 64 columns x 128 keys x all D/64 halves
        cuuint64_t dims[5] = {64, (cuuint64_t)p.Lcap, (cuuint64_t)(D / 64), (cuuint64_t)p.Hkv, (cuuint64_t)p.B};
        cuuint64_t str[4] = {(cuuint64_t)D * 2, 128, (cuuint64_t)p.Lcap * D * 2, (cuuint64_t)p.Hkv * p.Lcap * D * 2};
        cuuint32_t box[5] = {64, (cuuint32_t)kKeys, (cuuint32_t)(D / 64), 1, 1};
        if (!make_map_nd(&tmK, p.K, 5, dims, str, box)) return CTCSD_ERR_CUDA;
        if (!make_map_nd(&tmV, p.V, 5, dims, str, box)) return CTCSD_ERR_CUDA;
    }
    const size_t smem = (size_t)kRows * D * 2 + (size_t)kStages * 2 * kKeys * D * 2 +
                        ((size_t)kKeys * D * 2 >= (size_t)kRows * kKeys * 2 ? 0 : (size_t)kRows * kKeys * 2) + sizeof(AttnShared);
    auto kern = tree_attention_tc_kernel<D>;
    CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    CTCSD_CUDA_CHECK(h, launch_pdl(kern, dim3(qtiles * splits, p.Hkv, p.B), dim3(kThreads), smem, s, splits,
                                   tmQ, tmK, tmV, p, splits));
    h->launches++;
    return CTCSD_OK;
}

}  // namespace

bool tree_attention_tc_supported(const AttnParams& p) {
    const int grp = p.Hq / p.Hkv;
    if (grp < 1 || grp > kRows || (kRows % grp) != 0) return false;      // a query tile holds whole nodes
    if ((reinterpret_cast<uintptr_t>(p.Q) | reinterpret_cast<uintptr_t>(p.K) | reinterpret_cast<uintptr_t>(p.V)) & 15) return false;
    return p.D == 64 || p.D == 128;
}

int launch_tree_attention_tc(Handle* h, cudaStream_t s, const AttnParams& p) {
    if (!tree_attention_tc_supported(p)) return CTCSD_ERR_UNSUPPORTED;
    if (p.D == 64) return launch_tc<64>(h, s, p);
    return launch_tc<128>(h, s, p);
}

}  // namespace ctcsd
