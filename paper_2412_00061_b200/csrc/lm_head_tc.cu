// LM head on the 5th-generation tensor cores (tcgen05 + TMEM) with a fused row arg-max.
//
// y[m,v] = sum_h hn[m,h] * Wl[v,h] is computed as D[128 x Nt] = A[128 x K] * B[Nt x K]^T with
//   A = 128 rows of hn (rows past M are zero-filled by TMA), K-major, 128-byte swizzle,
//   B = Nt consecutive rows of Wl, K-major, 128-byte swizzle,
//   D = fp32 accumulator in tensor memory: lane = hn row, column = vocabulary row.
// The (vocabulary tile, row tile) units are dealt to the CTAs round-robin, so every weight is
// fetched from HBM once (row tiles that share a weight tile run at the same time and meet in L2); the kernel is a weight stream whose math hides behind the loads.
// Warp 0 issues TMA loads into a ring of shared-memory stages, warp 1 issues the MMAs, warps
// 2..17 read the accumulator back: four warps per quarter of the TMEM lanes (a warp may only
// read its own 32 lanes), each taking every fourth 32-column chunk of the tile, and keep the
// running arg-max of their row.  There are two accumulators.  With one row tile they alternate
// between consecutive units, so a unit's read-back runs under the next unit's MMAs; with more
// rows a stage carries two row tiles against one weight tile and each gets an accumulator.
// Each tile's winner is folded into the row's global maximum with one 64-bit atomic max on a
// packed (logit, complemented id) key, so ties go to the lower id; the CTA that finishes last
// unpacks the keys, clears them for the next call and runs the acceptance passes.
#include "lm_head_tc.cuh"
#include "tc_primitives.cuh"
#include "run_state.cuh"

#include <math.h>
#include <string.h>

namespace ctcsd {
namespace {

constexpr int kColSplit = kDraftColSplit;   // epilogue warps per TMEM lane quarter: each takes every 4th 32-column chunk
constexpr int kEpiWarps = 4 * kColSplit;
constexpr int kThreads = 64 + 32 * kEpiWarps;   // TMA warp, MMA warp, epilogue warps
constexpr int kBlockK = 64;                 // bf16 elements per 128-byte swizzle row
constexpr int kTileM = 128;
constexpr int kABytes = kTileM * 128;       // 16 KB
constexpr int kMaxStages = 8;
constexpr int kAccCols = 256;               // TMEM columns per accumulator (tiles are at most 256 wide)
constexpr int kTmemCols = 2 * kAccCols;

struct TcParams {
    int M;            // activation rows
    int V;            // vocabulary rows
    int num_k;        // K blocks of 64
    int Nt;           // vocabulary rows per tile (multiple of 16, <= 256)
    int n_tiles;      // vocabulary tiles
    int m_tiles;      // row tiles of 128
    int stages;
    int pair;         // 1: a stage holds two activation row tiles that share its weight tile
                      //    (both accumulators in use, one per row tile); 0: one row tile per stage,
                      //    the accumulators alternate between consecutive tiles
    int m_units;      // row tiles (pair = 0) or pairs of row tiles (pair = 1)
    int a_bytes;      // bytes of one K block of an activation tile: 128 rows, or 64 when M <= 64
    int atoms;        // K blocks (of 64 elements, one 128-byte swizzle row each) per stage: 1, or more when
                      // the hidden size is a multiple of 64 - one copy instruction then brings `atoms`
                      // blocks of a tile (a box over a [rows][K blocks][64] view of the tensor)
    int num_ks;       // stages per unit = ceil(num_k / atoms)
    unsigned long long* keys; // [m_tiles*128] packed (logit, id) maxima, zero between calls
    AcceptParams acc;
    unsigned* counter;
    int* out_argmax;          // [M]
    float* logits_dbg;        // null or [M][V]  (draft mode: [M][slots][V])
    int* status;
    // draft mode: W is [slots][V][H]; n_tiles = slots * tiles_per_slot
    int slots;
    int tiles_per_slot;
    int topk;                 // k: symbols kept per slot
    DraftPartial* part;       // [n_tiles][kColSplit][m_tiles*128] per-tile, per-column-share states
    const int* row_seq;       // [M] or null
    const float* blank_bias;  // [B] or null; added to class V-1 of every slot
    SampleNoise sn;           // LM head: noise added to the scaled logit before the arg-max (null: none)
    // LM head on more than one row tile: the rows of unused tree nodes are left out.  The
    // activation rows arrive packed (live rows only, sequence by sequence); row_map[r] is the tree
    // row of packed row r and row_map[row_map_len] the number of live rows, both written by the
    // kernel that precedes this one in the stream.  Null: every row is live and in place.
    const int* row_map;
    int row_map_len;
};

struct __align__(8) TcShared {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full[2];      // two accumulators: the epilogue of one tile runs under the next tile's MMAs
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    int abort_flag;
    int is_last;
    int never_set;      // stays zero: lets a drain wait run to its time limit after an abort
};

// MODE 0: LM head (row arg-max + acceptance).  MODE 1: draft head (W is a 3-D tensor
// [slots][V][H]; a vocabulary tile never crosses a slot; every epilogue thread folds its
// row's logits of the tile into an online (max, sum of exp, best-8) state and stores one
// state per (tile, row); a second kernel merges the tiles of every slot).
template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
lm_head_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, TcParams p) {
    extern __shared__ unsigned char dyn_raw[];
    // stage buffers need 1024-byte alignment for the 128-byte swizzle pattern
    const uint32_t raw_addr = tc::smem_u32(dyn_raw);
    unsigned char* dyn = dyn_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
    // a stage: activations [K block][row tile (two in pair mode)][a_bytes], then weights [K block][Nt x 128 bytes]
    const int a_blk = p.a_bytes * (1 + p.pair);             // one K block of the stage's activations
    const int a_all = a_blk * p.atoms;                      // activation bytes of a stage
    const int w_atom = p.Nt * 128;                          // one K block of the weight tile
    const int stage_bytes = a_all + w_atom * p.atoms;
    TcShared* sh = reinterpret_cast<TcShared*>(dyn + (size_t)p.stages * stage_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort_flag = &sh->abort_flag;

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], 1); }
        for (int a = 0; a < 2; ++a) { tc::mbar_init(&sh->tmem_full[a], 1); tc::mbar_init(&sh->tmem_empty[a], kEpiWarps); }
        sh->abort_flag = 0;
        sh->is_last = 0;
        sh->never_set = 0;
        tc::fence_barrier_init();
    }
    if (warp == 1) {
        tc::tmem_alloc(&sh->tmem_base, kTmemCols);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;
    int M = p.M, m_tiles = p.m_tiles, m_units = p.m_units;
    long long units = (long long)p.n_tiles * m_units;
    // CTA c takes units c, c + grid, c + 2 grid, ...: at any moment the CTAs then work on
    // neighbouring units, i.e. on the few row tiles of the same few weight tiles, so a weight tile
    // that several row tiles need is fetched from HBM once and found in L2 by the others.
    const int u_first = (int)blockIdx.x, u_step = (int)gridDim.x;
    int n_units = units > u_first ? (int)((units - u_first + u_step - 1) / u_step) : 0;

    // producer state (lane 0 of warp 0 only).  Stage `it` holds K blocks [ks * atoms, (ks+1) * atoms),
    // ks = it % num_ks, of unit u_first + (it / num_ks) * u_step; every CTA walks the K axis from its
    // own starting stage (and wraps), so that at any moment the CTAs ask L2 for different parts of
    // the shared activations.
    int total_it = n_units * p.num_ks;
    const int k_start = (int)(((long long)blockIdx.x * p.num_ks) / gridDim.x);
    const uint64_t pol_w = tc::policy_evict_first();
    const uint64_t pol_a = tc::policy_evict_last();
    auto load_stage = [&](int it, bool do_w, bool do_a) {
        const int u = u_first + (it / p.num_ks) * u_step, kb = it - (it / p.num_ks) * p.num_ks;
        const int nt = u / m_units, mu = u - nt * m_units;
        const int s = it % p.stages;
        unsigned char* a_dst = dyn + (size_t)s * stage_bytes;
        int kq = kb + k_start;
        if (kq >= p.num_ks) kq -= p.num_ks;
        // K blocks past the end of the hidden axis (the last stage when atoms does not divide num_k)
        // lie outside the tensor and arrive as zeros
        if (do_w) {
            tc::mbar_arrive_expect_tx(&sh->full[s], (uint32_t)stage_bytes);
            if constexpr (MODE == 0) {
                if (p.atoms == 1) tc::tma_load_2d(a_dst + a_all, &tmW, &sh->full[s], kq * kBlockK, nt * p.Nt, pol_w);
                else tc::tma_load_3d(a_dst + a_all, &tmW, &sh->full[s], 0, nt * p.Nt, kq * p.atoms, pol_w);
            } else {
                const int t = nt / p.tiles_per_slot, ntl = nt - t * p.tiles_per_slot;
                if (p.atoms == 1) tc::tma_load_3d(a_dst + a_all, &tmW, &sh->full[s], kq * kBlockK, ntl * p.Nt, t, pol_w);
                else tc::tma_load_4d(a_dst + a_all, &tmW, &sh->full[s], 0, ntl * p.Nt, kq * p.atoms, t, pol_w);
            }
        }
        if (do_a) {
            // one box: in pair mode it is 256 rows high and brings both row tiles (rows past the last
            // activation row read as zeros)
            const int row0 = (p.pair ? 2 * mu : mu) * kTileM;
            if (p.atoms == 1) tc::tma_load_2d(a_dst, &tmA, &sh->full[s], kq * kBlockK, row0, pol_a);
            else tc::tma_load_3d(a_dst, &tmA, &sh->full[s], 0, row0, kq * p.atoms, pol_a);
        }
    };
    // The weights are never written by any kernel: their tiles of the first stages are requested
    // before this kernel waits for its predecessor in the stream.
    int pre = 0;
    if (warp == 0 && lane == 0) {
        tc::prefetch_tensormap(&tmA);
        tc::prefetch_tensormap(&tmW);
        // (with packed rows the units are known only once the live-row count can be read)
        if (p.row_map == nullptr) {
            pre = total_it < p.stages ? total_it : p.stages;
            for (int it = 0; it < pre; ++it) load_stage(it, true, false);
        }
    }
    // barriers and tensor memory are set up; the activations may come from the preceding kernel
    pdl_wait();
    pdl_trigger();
    if (p.row_map != nullptr) {
        // only the row tiles that hold live rows are units of work
        M = p.row_map[p.row_map_len];
        M = M < 0 ? 0 : (M > p.M ? p.M : M);
        m_tiles = (M + kTileM - 1) / kTileM;
        m_units = p.pair ? (m_tiles + 1) / 2 : m_tiles;
        units = (long long)p.n_tiles * m_units;
        n_units = units > u_first ? (int)((units - u_first + u_step - 1) / u_step) : 0;
        total_it = n_units * p.num_ks;
    }

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            for (int it = 0; it < pre; ++it) load_stage(it, false, true);
            int it = pre;
            bool ok = true;
            // Stages are refilled two at a time: the two weight boxes then ask for adjacent 128-byte
            // pieces of the same rows close together in time, which DRAM serves better than the
            // same requests a stage apart (measured: 4 us of 70 on the 7B LM head).
            const int group = p.stages >= 4 ? 2 : 1;
            while (it < total_it && ok) {
                const int cnt = total_it - it < group ? total_it - it : group;
                for (int j = 0; j < cnt; ++j) {
                    const int s = (it + j) % p.stages;
                    const uint32_t ph = (uint32_t)((it + j) / p.stages) & 1u;
                    if (!tc::mbar_wait(&sh->empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                }
                if (!ok) break;
                for (int j = 0; j < cnt; ++j) load_stage(it + j, true, false);
                for (int j = 0; j < cnt; ++j) load_stage(it + j, false, true);
                it += cnt;
            }
            if (!ok) {
                if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 1);
                *abort_flag = 1;
                // let copies that are still in flight land before the CTA gives its memory back
                for (int back = 1; back <= p.stages && back <= it; ++back) {
                    const int j = it - back;
                    tc::mbar_wait(&sh->full[j % p.stages], (uint32_t)(j / p.stages) & 1u, &sh->never_set, 1ll << 24);
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_bf16_f32(kTileM, p.Nt);
            int it = 0, ucount = 0;
            bool ok = true;
            for (int u = u_first; ucount < n_units && ok; u += u_step, ++ucount) {
                const int acc = p.pair ? 0 : (ucount & 1);            // barrier pair that guards this unit
                const bool second = p.pair && 2 * (u % m_units) + 1 < m_tiles;   // the pair's second row tile exists
                const uint32_t acc_ph = (uint32_t)(p.pair ? ucount : (ucount >> 1)) & 1u;
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kAccCols);
                if (!tc::mbar_wait(&sh->tmem_empty[acc], acc_ph ^ 1u, abort_flag)) { ok = false; break; }
                tc::tc_fence_after_sync();
                for (int kb = 0; kb < p.num_ks; ++kb, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
                    if (!tc::mbar_wait(&sh->full[s], ph, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after_sync();
                    const uint32_t a_addr = tc::smem_u32(dyn + (size_t)s * stage_bytes);
                    // which K blocks the stage holds decides nothing here except how many are real:
                    // the rotated order only permutes the terms of the sum
                    int kq = kb + k_start;
                    if (kq >= p.num_ks) kq -= p.num_ks;
                    for (int j = 0; j < p.atoms; ++j) {
                        if (kq * p.atoms + j >= p.num_k) break;          // zero blocks past the hidden axis
                        const uint64_t adesc = tc::smem_desc_k_sw128(a_addr + (uint32_t)(j * a_blk));
                        const uint64_t bdesc = tc::smem_desc_k_sw128(a_addr + (uint32_t)(a_all + j * w_atom));
#pragma unroll
                        for (int k = 0; k < kBlockK / 16; ++k) {
                            // advancing 16 bf16 along K = 32 bytes = 2 descriptor address units
                            tc::mma_bf16_ss(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | j | k) != 0 ? 1u : 0u);
                        }
                        if (second) {                        // the second row tile against the same weights
                            const uint64_t adesc1 = tc::smem_desc_k_sw128(a_addr + (uint32_t)(j * a_blk + p.a_bytes));
#pragma unroll
                            for (int k = 0; k < kBlockK / 16; ++k)
                                tc::mma_bf16_ss(d_tmem + kAccCols, adesc1 + 2 * k, bdesc + 2 * k, idesc, (kb | j | k) != 0 ? 1u : 0u);
                        }
                    }
                    tc::mma_commit(&sh->empty[s]);          // frees the stage once these MMAs have read it
                }
                if (ok) tc::mma_commit(&sh->tmem_full[acc]);
            }
            if (!ok) {
                if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 2);
                *abort_flag = 1;
            }
        }
    } else {
        // ---------------- epilogue ----------------
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int cs = (warp - 2) >> 2;               // which share of the tile's columns
        const bool few = MODE == 1 && p.topk <= 4;    // draft mode: a four-entry list is enough
        const int row_in_tile = q * 32 + lane;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        int ucount = 0;
        bool ok = true;
        for (int u = u_first; ucount < n_units && ok; u += u_step, ++ucount) {
            const int nt = u / m_units, mu = u - nt * m_units;
            // draft mode: tile nt is tile ntl of slot t
            const int t = MODE == 1 ? nt / p.tiles_per_slot : 0;
            const int n0 = (MODE == 1 ? nt - t * p.tiles_per_slot : nt) * p.Nt;
            const int acc = p.pair ? 0 : (ucount & 1);
            const uint32_t acc_ph = (uint32_t)(p.pair ? ucount : (ucount >> 1)) & 1u;
            if (!tc::mbar_wait_idle(&sh->tmem_full[acc], acc_ph, abort_flag)) { ok = false; break; }
            tc::tc_fence_after_sync();
            for (int h = 0; h <= p.pair; ++h) {               // pair mode: accumulator h holds row tile 2*mu + h
            const int mt = p.pair ? 2 * mu + h : mu;
            const int row = mt * kTileM + row_in_tile;
            // the tree row this (packed) row stands for: debug logits and noise are addressed by it
            const int orow = (MODE == 0 && p.row_map != nullptr && row < M) ? p.row_map[row] : row;
            float bias = 0.f;
            if (MODE == 1 && p.blank_bias != nullptr && row < p.M) bias = p.blank_bias[p.row_seq ? p.row_seq[row] : row];
            const uint32_t lane_addr = lane_base + (uint32_t)((p.pair ? h : acc) * kAccCols);
            float best = -INFINITY;
            int best_idx = 0x7fffffff;
            const float* noise_row = nullptr;                 // sampling acceptance: the row's Gumbel noise
            if (MODE == 0 && p.sn.noise != nullptr && row < M) {
                int d = p.sn.depth[orow];
                d = d < 0 ? 0 : (d >= p.sn.rows_per_seq ? p.sn.rows_per_seq - 1 : d);
                noise_row = p.sn.noise + ((size_t)(orow / p.sn.max_nodes) * p.sn.rows_per_seq + d) * (size_t)p.V;
            }
            RunState st;
            if constexpr (MODE == 1) st.init();
            // a warp whose 32 rows lie past the last activation row has nothing to read
            const int c_end = (mt * kTileM + q * 32 < M) ? p.Nt : 0;
            for (int c0 = cs * 32; c0 < c_end; c0 += 32 * kColSplit) {
                uint32_t r[32];
                if (c0 + 32 <= p.Nt) {
                    tc::tmem_ld32(lane_addr + (uint32_t)c0, r);
                } else {                                  // Nt is a multiple of 16: 16-column tail
                    uint32_t r16[16];
                    tc::tmem_ld16(lane_addr + (uint32_t)c0, r16);
#pragma unroll
                    for (int j = 0; j < 16; ++j) { r[j] = r16[j]; r[16 + j] = 0xff800000u; }
                }
                tc::tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    float v = __uint_as_float(r[j]);
                    const int col = n0 + c0 + j;
                    if (col < p.V && c0 + j < p.Nt) {
                        if constexpr (MODE == 0) {
                            if (p.logits_dbg != nullptr && row < M) p.logits_dbg[(size_t)orow * p.V + col] = v;
                            if (noise_row != nullptr) v = __fmaf_rn(v, p.sn.inv_temp, __ldg(noise_row + col));
                            if (v > best) { best = v; best_idx = col; }
                        } else {
                            if (col == p.V - 1) v += bias;
                            if (p.logits_dbg != nullptr && row < p.M)
                                p.logits_dbg[((size_t)row * p.slots + t) * p.V + col] = v;
                            if (few) st.push_n<4>(v, col); else st.push(v, col);
                        }
                    }
                }
            }
            if (h == p.pair) {                                // the last accumulator of the unit has been read
                tc::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(&sh->tmem_empty[acc]);
            }
            if constexpr (MODE == 1) {
                // (the second row tile of the last pair does not exist when the tile count is odd)
                if (mt < p.m_tiles) st.store(p.part + ((size_t)nt * kColSplit + cs) * (p.m_tiles * kTileM) + row);
            } else {
            // fold this tile's winner into the row's global maximum: larger logit first, equal
            // logits -> lower id (the id is stored complemented in the low word)
            if (row < M && best_idx != 0x7fffffff) {
                const unsigned u = __float_as_uint(best);
                const unsigned sortable = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
                atomicMax(p.keys + row, ((unsigned long long)sortable << 32) | (0xffffffffu - (unsigned)best_idx));
            }
            }
            }
        }
        if (!ok && lane == 0) {
            if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 3);
            *abort_flag = 1;
        }
    }

    // ---------------- teardown and cross-CTA reduction ----------------
    __threadfence();
    tc::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc::tc_fence_after_sync();
        tc::tmem_dealloc(tmem_base, kTmemCols);
    }
    if constexpr (MODE == 1) return;                 // the tiles are merged by draft_tc_merge_kernel
    if (tid == 0) {
        unsigned t = atomicAdd(p.counter, 1u);
        sh->is_last = (t == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!sh->is_last) return;
    __threadfence();
    const bool good = sh->abort_flag == 0;
    for (int row = tid; row < M; row += kThreads) {
        const unsigned long long key = __ldcg(p.keys + row);
        const int orow = p.row_map != nullptr ? p.row_map[row] : row;
        if (good) p.out_argmax[orow] = (int)(0xffffffffu - (unsigned)(key & 0xffffffffull));
        p.keys[row] = 0ull;
    }
    __syncthreads();
    // the pipeline stages are idle now: their shared memory serves as the acceptance scratch
    if (good)
    {
        int aw = (int)(((size_t)p.stages * stage_bytes) / (kAcceptScratchInts * sizeof(int)));
        aw = aw < kThreads / 32 ? aw : kThreads / 32;          // warps the stage memory can serve (>= 1)
        if (warp < aw)
            for (int b = warp; b < p.acc.B; b += aw)
                accept_warp(p.acc, b, lane, reinterpret_cast<int*>(dyn) + warp * kAcceptScratchInts);
    }
    if (tid == 0) *p.counter = 0u;
}

// Packs the activation rows of the live tree nodes densely, sequence by sequence, for the LM head on
// more than one row tile: the rows of unused nodes (a tree rarely fills its budget) then cost
// neither tensor-core work nor an epilogue.  One CTA per tree row (node i of sequence b).  Writes
// row_map (packed row -> tree row), the live-row count behind it, and -1 as the arg-max of every
// unused node.
__global__ void __launch_bounds__(128) lm_pack_rows_kernel(const uint4* hn, const int* n_nodes, int B, int max_nodes,
                                                           int chunks, uint4* packed, int* row_map, int row_map_len,
                                                           int* out_argmax) {
    __shared__ int s_part[4];
    const int i = blockIdx.x, b = blockIdx.y, tid = threadIdx.x;
    pdl_wait();                      // the node counts and the activations come from preceding kernels
    pdl_trigger();
    auto count = [&](int q) { const int n = n_nodes[q]; return n < 0 ? 0 : (n > max_nodes ? max_nodes : n); };
    int before = 0;                                   // live rows of the sequences before this one
    for (int q = tid; q < b; q += 128) before += count(q);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
    if ((tid & 31) == 0) s_part[tid >> 5] = before;
    __syncthreads();
    const int off = s_part[0] + s_part[1] + s_part[2] + s_part[3];
    const int n = count(b);
    const int orow = b * max_nodes + i;
    if (b == B - 1 && i == 0 && tid == 0) row_map[row_map_len] = off + n;
    if (i >= n) {
        if (tid == 0) out_argmax[orow] = -1;
        return;
    }
    const int prow = off + i;
    if (tid == 0) row_map[prow] = orow;
    const uint4* src = hn + (size_t)orow * chunks;
    uint4* dst = packed + (size_t)prow * chunks;
    for (int c = tid; c < chunks; c += 128) dst[c] = src[c];
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

// 2-D bf16 tensor [rows][cols] (cols contiguous), box = [box_rows][64 cols], 128-byte swizzle,
// out-of-range elements read as zero.
bool make_map(CUtensorMap* map, const void* base, long long rows, long long cols, int box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)kBlockK, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// 3-D bf16 tensor [slots][rows][cols] (cols contiguous), box = [1][box_rows][64 cols], 128-byte
// swizzle; rows past the end of a slot read as zero.
bool make_map3(CUtensorMap* map, const void* base, long long slots, long long rows, long long cols, int box_rows) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)cols, (cuuint64_t)rows, (cuuint64_t)slots};
    cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)cols * 2 * (cuuint64_t)rows};
    cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The same tensors seen as [rows][K blocks][64 elements] (and [slots][rows][K blocks][64]), which
// needs the hidden size to be a multiple of 64: a box of `atoms` K blocks x box_rows rows x 64
// elements lands in shared memory as `atoms` consecutive 128-byte-swizzled K-major tiles, so one
// copy instruction does the work of `atoms` (each instruction costs the copy engine a fixed few
// hundred nanoseconds whatever its size, which is what bounds a stream of small boxes), and DRAM
// is asked for atoms x 128 contiguous bytes of every row at once.
bool make_map_kblocks(CUtensorMap* map, const void* base, long long rows, long long cols, int box_rows, int atoms) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn || cols % kBlockK != 0) return false;
    cuuint64_t dims[3] = {(cuuint64_t)kBlockK, (cuuint64_t)rows, (cuuint64_t)(cols / kBlockK)};
    cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)kBlockK * 2};
    cuuint32_t box[3] = {(cuuint32_t)kBlockK, (cuuint32_t)box_rows, (cuuint32_t)atoms};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool make_map3_kblocks(CUtensorMap* map, const void* base, long long slots, long long rows, long long cols, int box_rows,
                       int atoms) {
    EncodeTiledFn fn = get_encode_fn();
    if (!fn || cols % kBlockK != 0) return false;
    cuuint64_t dims[4] = {(cuuint64_t)kBlockK, (cuuint64_t)rows, (cuuint64_t)(cols / kBlockK), (cuuint64_t)slots};
    cuuint64_t strides[3] = {(cuuint64_t)cols * 2, (cuuint64_t)kBlockK * 2, (cuuint64_t)cols * 2 * (cuuint64_t)rows};
    cuuint32_t box[4] = {(cuuint32_t)kBlockK, (cuuint32_t)box_rows, (cuuint32_t)atoms, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// K blocks per stage: as many (up to 4) as still leave `min_stages` stages in shared memory; 1
// when the hidden size is not a multiple of 64 (the last K block is then partial and only the
// plain 2-D view reads it correctly).
int choose_atoms(int H, int num_k, int one_block_bytes, int min_stages) {
    if (H % kBlockK != 0) return 1;
    const int budget = 220 * 1024 - (int)sizeof(TcShared) - 1024;
    int atoms = 1;
    while (atoms < 4 && atoms * 2 <= num_k && budget / (one_block_bytes * atoms * 2) >= min_stages) atoms *= 2;
    return atoms;
}

struct DraftMergeParams {
    const DraftPartial* part;     // [slots * tiles_per_slot * kColSplit][mpad]
    int M, mpad, slots, tiles_per_slot, k;
    int* out_topk_id; float* out_topk_lp; float* out_lse;
};

// One CTA of sixteen warps per (activation row, slot): every thread folds its share of the slot's
// per-tile states (about one each at a 32000-word vocabulary: folding a state is a chain of list
// insertions), the warps combine theirs, and the first warp combines the sixteen results into the
// log-sum-exp and the top-k of the row.
constexpr int kMergeThreads = 512;
__global__ void __launch_bounds__(kMergeThreads) draft_tc_merge_kernel(DraftMergeParams p) {
    __shared__ DraftPartial s_warp[kMergeThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long pair = blockIdx.x;
    pdl_wait();
    pdl_trigger();
    const int m = (int)(pair / p.slots), t = (int)(pair - (long long)m * p.slots);
    RunState fs;
    fs.init();
    const int entries = p.tiles_per_slot * kColSplit;          // per tile: one state per column share
    for (int e = threadIdx.x; e < entries; e += kMergeThreads)
        fs.absorb(load_partial_cg(p.part + ((size_t)t * entries + e) * p.mpad + m));
    warp_combine(fs);
    if (lane == 0) fs.store(&s_warp[warp]);
    __syncthreads();
    if (warp != 0) return;
    fs.init();
    if (lane < kMergeThreads / 32) fs.absorb(s_warp[lane]);
    warp_combine(fs);
    if (lane == 0) {
        const float lse = fs.mx + logf(fs.sum);
        p.out_lse[(size_t)m * p.slots + t] = lse;
#pragma unroll
        for (int j = 0; j < kTopSlots; ++j) {
            if (j < p.k) {
                const size_t o = ((size_t)m * p.slots + t) * p.k + j;
                p.out_topk_id[o] = fs.id[j];
                p.out_topk_lp[o] = fs.val[j] - lse;
            }
        }
    }
}

}  // namespace

int draft_tc_tile_rows(int classes) {
    if (classes >= 224) return 224;
    return (classes + 15) / 16 * 16;
}

bool draft_head_tc_supported(const Handle* h, int M) {
    const ctcsd_config& c = h->cfg;
    return c.dtype == CTCSD_DTYPE_BF16 && c.H >= 64 && c.V + 1 >= 16 && M > 8 && h->lay.tc_part_bytes > 0;
}

int launch_draft_head_tc(Handle* h, cudaStream_t stream, int M, const void* x, const void* Wd, const int* row_seq,
                         const float* blank_bias, int* out_topk_id, float* out_topk_lp, float* out_lse,
                         float* out_logits_dbg) {
    const ctcsd_config& c = h->cfg;
    if (!draft_head_tc_supported(h, M)) return CTCSD_ERR_UNSUPPORTED;
    TcParams p;
    memset(&p, 0, sizeof(p));
    p.M = M;
    p.V = c.V + 1;                                   // classes per slot, blank included
    p.num_k = (c.H + kBlockK - 1) / kBlockK;
    p.m_tiles = (M + kTileM - 1) / kTileM;
    p.Nt = draft_tc_tile_rows(p.V);
    p.slots = c.T;
    p.topk = c.k;
    p.tiles_per_slot = (p.V + p.Nt - 1) / p.Nt;
    p.n_tiles = p.slots * p.tiles_per_slot;
    const size_t need = sizeof(DraftPartial) * (size_t)p.n_tiles * kColSplit * p.m_tiles * kTileM;
    if (need > h->lay.tc_part_bytes) return CTCSD_ERR_WORKSPACE;
    // up to 64 rows: only the lower half of the activation tile is loaded (see launch_lm_head_tc)
    p.a_bytes = (M <= 64 && p.Nt * 128 >= kABytes / 2) ? kABytes / 2 : kABytes;
    // One row tile per stage, the two accumulators alternating so that a tile's epilogue runs under the
    // next tile's products.  (Two row tiles per weight stage, as in the LM head, were measured on the
    // 70B shape with 2048 rows: 7.5 ms against 7.1 ms - the products already take the shared-memory
    // bandwidth that their operands need, and the epilogue then runs with the tensor core idle.)
    p.pair = 0;
    p.m_units = p.pair ? (p.m_tiles + 1) / 2 : p.m_tiles;
    // (two stages of two K blocks stream faster here than four stages of one: measured on the 70B shape)
    p.atoms = choose_atoms(c.H, p.num_k, p.a_bytes * (1 + p.pair) + p.Nt * 128, 2);
    p.num_ks = (p.num_k + p.atoms - 1) / p.atoms;
    const int stage_bytes = (p.a_bytes * (1 + p.pair) + p.Nt * 128) * p.atoms;
    int stages = (int)((220 * 1024 - (int)sizeof(TcShared) - 1024) / stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return CTCSD_ERR_UNSUPPORTED;
    p.stages = stages;
    p.part = reinterpret_cast<DraftPartial*>(h->ws + h->lay.tc_part_off);
    p.row_seq = row_seq;
    p.blank_bias = blank_bias;
    p.logits_dbg = out_logits_dbg;
    p.status = status_ptr(h);

    CUtensorMap tmA, tmW;
    const int a_box_rows = p.a_bytes / 128 * (1 + p.pair);
    if (p.atoms == 1) {
        if (!make_map(&tmA, x, M, c.H, a_box_rows)) return CTCSD_ERR_CUDA;
        if (!make_map3(&tmW, Wd, p.slots, p.V, c.H, p.Nt)) return CTCSD_ERR_CUDA;
    } else {
        if (!make_map_kblocks(&tmA, x, M, c.H, a_box_rows, p.atoms)) return CTCSD_ERR_CUDA;
        if (!make_map3_kblocks(&tmW, Wd, p.slots, p.V, c.H, p.Nt, p.atoms)) return CTCSD_ERR_CUDA;
    }
    const size_t smem = (size_t)stages * stage_bytes + sizeof(TcShared) + 1024;
    CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(lm_head_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    long long units = (long long)p.n_tiles * p.m_units;
    int grid = (int)(units < h->num_sms ? units : h->num_sms);
    CTCSD_CUDA_CHECK(h, launch_pdl(lm_head_tc_kernel<1>, dim3(grid), dim3(kThreads), smem, stream, 1, tmA, tmW, p));
    CTCSD_LAUNCH_CHECK(h);

    DraftMergeParams mp;
    mp.part = p.part;
    mp.M = M; mp.mpad = p.m_tiles * kTileM; mp.slots = p.slots; mp.tiles_per_slot = p.tiles_per_slot; mp.k = c.k;
    mp.out_topk_id = out_topk_id; mp.out_topk_lp = out_topk_lp; mp.out_lse = out_lse;
    const long long pairs = (long long)M * p.slots;           // one CTA each
    CTCSD_CUDA_CHECK(h, launch_pdl(draft_tc_merge_kernel, dim3((unsigned)pairs), dim3(kMergeThreads), 0, stream, 1, mp));
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}

bool lm_head_tc_supported(const Handle* h) {
    const ctcsd_config& c = h->cfg;
    return c.dtype == CTCSD_DTYPE_BF16 && c.H % 8 == 0 && c.H >= 64 && c.V >= 16;
}

int launch_lm_head_tc(Handle* h, cudaStream_t stream, int M, const void* hn, const void* Wl,
                      int* out_argmax, float* out_logits_dbg, const AcceptParams& acc, const SampleNoise& sn) {
    const ctcsd_config& c = h->cfg;
    if (!lm_head_tc_supported(h)) return CTCSD_ERR_UNSUPPORTED;

    TcParams p;
    memset(&p, 0, sizeof(p));
    p.M = M;
    p.V = c.V;
    p.num_k = (c.H + kBlockK - 1) / kBlockK;
    p.m_tiles = (M + kTileM - 1) / kTileM;
    // vocabulary rows per tile: spread the 16-row groups evenly over the SMs, at most 256 rows
    const int groups = (c.V + 15) / 16;
    int per_sm = (groups + h->num_sms - 1) / h->num_sms;
    int rounds = (per_sm + 15) / 16;
    int g_per_tile = (per_sm + rounds - 1) / rounds;
    p.Nt = 16 * g_per_tile;
    // Two or more row tiles: there are many more units than SMs, so the tiles need not be cut to
    // the SM count; the widest tile gives the most flops per copy instruction and per weight byte.
    if (p.m_tiles >= 2 && c.V >= 256) p.Nt = 256;
    p.n_tiles = (c.V + p.Nt - 1) / p.Nt;
    if (p.m_tiles * kTileM > h->lay.lm_key_count) return CTCSD_ERR_WORKSPACE;
    // With at most 64 rows only the lower half of the 128-row activation tile is loaded.  The
    // tensor core still reads 128 rows: the upper 64 come from the first 8 KB of the stage's
    // weight tile (so that must be at least that large), and the accumulator rows they produce
    // belong to no activation row and are never looked at.
    const bool half_a = M <= 64 && p.Nt * 128 >= kABytes / 2;
    p.a_bytes = half_a ? kABytes / 2 : kABytes;
    // Two or more row tiles: a weight stage feeds two of them, which halves the shared-memory fill
    // per flop (with one row tile per 28 KB weight stage the tensor core waits for L2).
    p.pair = p.m_tiles >= 2 ? 1 : 0;
    p.m_units = p.pair ? (p.m_tiles + 1) / 2 : p.m_tiles;
    p.atoms = choose_atoms(c.H, p.num_k, p.a_bytes * (1 + p.pair) + p.Nt * 128, 3);
    p.num_ks = (p.num_k + p.atoms - 1) / p.atoms;
    const int stage_bytes = (p.a_bytes * (1 + p.pair) + p.Nt * 128) * p.atoms;
    int stages = (int)((220 * 1024 - (int)sizeof(TcShared) - 1024) / stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return CTCSD_ERR_UNSUPPORTED;
    p.stages = stages;
    p.keys = reinterpret_cast<unsigned long long*>(h->ws + h->lay.lm_key_off);
    p.acc = acc;
    p.sn = sn;
    p.counter = counter_ptr(h) + 1;
    p.out_argmax = out_argmax;
    p.logits_dbg = out_logits_dbg;
    p.status = status_ptr(h);

    // More than one row tile: the live rows are packed first (the rows of unused nodes are skipped).
    const void* a_rows = hn;
    long long a_row_count = M;
    if (p.m_tiles >= 2 && h->lay.lm_rowmap_off != h->lay.lm_rows_off && acc.n_nodes != nullptr) {
        uint4* packed = reinterpret_cast<uint4*>(h->ws + h->lay.lm_rows_off);
        int* row_map = reinterpret_cast<int*>(h->ws + h->lay.lm_rowmap_off);
        CTCSD_CUDA_CHECK(h, launch_pdl(lm_pack_rows_kernel, dim3(c.max_nodes, c.B), dim3(128), 0, stream, 1,
                                       static_cast<const uint4*>(hn), acc.n_nodes, c.B, c.max_nodes, c.H / 8, packed,
                                       row_map, h->lay.lm_key_count, out_argmax));
        CTCSD_LAUNCH_CHECK(h);
        p.row_map = row_map;
        p.row_map_len = h->lay.lm_key_count;
        a_rows = packed;
        a_row_count = h->lay.lm_key_count;
    }
    CUtensorMap tmA, tmW;
    const int a_box_rows = p.a_bytes / 128 * (1 + p.pair);
    if (p.atoms == 1) {
        if (!make_map(&tmA, a_rows, a_row_count, c.H, a_box_rows)) return CTCSD_ERR_CUDA;
        if (!make_map(&tmW, Wl, c.V, c.H, p.Nt)) return CTCSD_ERR_CUDA;
    } else {
        if (!make_map_kblocks(&tmA, a_rows, a_row_count, c.H, a_box_rows, p.atoms)) return CTCSD_ERR_CUDA;
        if (!make_map_kblocks(&tmW, Wl, c.V, c.H, p.Nt, p.atoms)) return CTCSD_ERR_CUDA;
    }

    const size_t smem = (size_t)stages * stage_bytes + sizeof(TcShared) + 1024;
    CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(lm_head_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    long long units = (long long)p.n_tiles * p.m_units;
    int grid = (int)(units < h->num_sms ? units : h->num_sms);
    CTCSD_CUDA_CHECK(h, launch_pdl(lm_head_tc_kernel<0>, dim3(grid), dim3(kThreads), smem, stream, 1, tmA, tmW, p));
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}

}  // namespace ctcsd
