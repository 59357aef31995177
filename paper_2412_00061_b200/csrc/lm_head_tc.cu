// LM head on the 5th-generation tensor cores (tcgen05 + TMEM) with a fused row arg-max.
//
// y[m,v] = sum_h hn[m,h] * Wl[v,h] is computed as D[128 x Nt] = A[128 x K] * B[Nt x K]^T with
//   A = 128 rows of hn (rows past M are zero-filled by TMA), K-major, 128-byte swizzle,
//   B = Nt consecutive rows of Wl, K-major, 128-byte swizzle,
//   D = fp32 accumulator in tensor memory: lane = hn row, column = vocabulary row.
// Each CTA owns a contiguous range of (vocabulary tile, row tile) units, so every weight is
// fetched from HBM once; the kernel is a weight stream whose math hides behind the loads.
// Warp 0 issues TMA loads into a ring of shared-memory stages, warp 1 issues the MMAs,
// warps 2..5 read the accumulator back (each warp its own 32 TMEM lanes) and keep the
// running arg-max of their row.  Each tile's winner is folded into the row's global maximum
// with one 64-bit atomic max on a packed (logit, complemented id) key, so ties go to the
// lower id; the CTA that finishes last unpacks the keys, clears them for the next call and
// runs the greedy acceptance walk.
#include "lm_head_tc.cuh"
#include "tc_primitives.cuh"

#include <math.h>

namespace ctcsd {
namespace {

constexpr int kThreads = 192;
constexpr int kBlockK = 64;                 // bf16 elements per 128-byte swizzle row
constexpr int kTileM = 128;
constexpr int kABytes = kTileM * 128;       // 16 KB
constexpr int kMaxStages = 8;

struct TcParams {
    int M;            // activation rows
    int V;            // vocabulary rows
    int num_k;        // K blocks of 64
    int Nt;           // vocabulary rows per tile (multiple of 16, <= 256)
    int n_tiles;      // vocabulary tiles
    int m_tiles;      // row tiles of 128
    int stages;
    unsigned long long* keys; // [m_tiles*128] packed (logit, id) maxima, zero between calls
    AcceptParams acc;
    unsigned* counter;
    int* out_argmax;          // [M]
    float* logits_dbg;        // null or [M][V]
    int* status;
};

struct __align__(8) TcShared {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full;
    uint64_t tmem_empty;
    uint32_t tmem_base;
    int abort_flag;
    int is_last;
    int never_set;      // stays zero: lets a drain wait run to its time limit after an abort
};

__global__ void __launch_bounds__(kThreads, 1)
lm_head_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmW, TcParams p) {
    extern __shared__ unsigned char dyn_raw[];
    // stage buffers need 1024-byte alignment for the 128-byte swizzle pattern
    const uint32_t raw_addr = tc::smem_u32(dyn_raw);
    unsigned char* dyn = dyn_raw + ((1024u - (raw_addr & 1023u)) & 1023u);
    const int stage_bytes = kABytes + p.Nt * 128;
    TcShared* sh = reinterpret_cast<TcShared*>(dyn + (size_t)p.stages * stage_bytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort_flag = &sh->abort_flag;

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) { tc::mbar_init(&sh->full[s], 1); tc::mbar_init(&sh->empty[s], 1); }
        tc::mbar_init(&sh->tmem_full, 1);
        tc::mbar_init(&sh->tmem_empty, 4);
        sh->abort_flag = 0;
        sh->is_last = 0;
        sh->never_set = 0;
        tc::fence_barrier_init();
    }
    if (warp == 1) {
        tc::tmem_alloc(&sh->tmem_base, 256);
        tc::tmem_relinquish();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tmem_base = sh->tmem_base;
    const long long units = (long long)p.n_tiles * p.m_tiles;
    const int u0 = (int)(units * blockIdx.x / gridDim.x);
    const int u1 = (int)(units * (blockIdx.x + 1) / gridDim.x);

    // producer state (lane 0 of warp 0 only).  Stage `it` holds K block it % num_k of unit
    // u0 + it / num_k; every CTA walks the K axis from its own starting block (and wraps), so that
    // at any moment the CTAs ask L2 for different parts of the shared activations.
    const int total_it = (u1 - u0) * p.num_k;
    const int k_start = (int)(((long long)blockIdx.x * p.num_k) / gridDim.x);
    const uint64_t pol_w = tc::policy_evict_first();
    const uint64_t pol_a = tc::policy_evict_last();
    auto load_stage = [&](int it, bool do_w, bool do_a) {
        const int u = u0 + it / p.num_k, kb = it - (it / p.num_k) * p.num_k;
        const int nt = u / p.m_tiles, mt = u - nt * p.m_tiles;
        const int s = it % p.stages;
        unsigned char* a_dst = dyn + (size_t)s * stage_bytes;
        int kq = kb + k_start;
        if (kq >= p.num_k) kq -= p.num_k;
        if (do_w) {
            tc::mbar_arrive_expect_tx(&sh->full[s], (uint32_t)stage_bytes);
            tc::tma_load_2d(a_dst + kABytes, &tmW, &sh->full[s], kq * kBlockK, nt * p.Nt, pol_w);
        }
        if (do_a) tc::tma_load_2d(a_dst, &tmA, &sh->full[s], kq * kBlockK, mt * kTileM, pol_a);
    };
    // The weights are never written by any kernel: their tiles of the first stages are requested
    // before this kernel waits for its predecessor in the stream.
    int pre = 0;
    if (warp == 0 && lane == 0) {
        tc::prefetch_tensormap(&tmA);
        tc::prefetch_tensormap(&tmW);
        pre = total_it < p.stages ? total_it : p.stages;
        for (int it = 0; it < pre; ++it) load_stage(it, true, false);
    }
    // barriers and tensor memory are set up; the activations may come from the preceding kernel
    pdl_wait();
    pdl_trigger();

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            for (int it = 0; it < pre; ++it) load_stage(it, false, true);
            int it = pre;
            bool ok = true;
            for (; it < total_it; ++it) {
                const int s = it % p.stages;
                const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
                if (!tc::mbar_wait(&sh->empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                load_stage(it, true, true);
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
            for (int u = u0; u < u1 && ok; ++u, ++ucount) {
                if (!tc::mbar_wait(&sh->tmem_empty, ((uint32_t)ucount & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                tc::tc_fence_after_sync();
                for (int kb = 0; kb < p.num_k; ++kb, ++it) {
                    const int s = it % p.stages;
                    const uint32_t ph = (uint32_t)(it / p.stages) & 1u;
                    if (!tc::mbar_wait(&sh->full[s], ph, abort_flag)) { ok = false; break; }
                    tc::tc_fence_after_sync();
                    const uint32_t a_addr = tc::smem_u32(dyn + (size_t)s * stage_bytes);
                    const uint64_t adesc = tc::smem_desc_k_sw128(a_addr);
                    const uint64_t bdesc = tc::smem_desc_k_sw128(a_addr + kABytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k) {
                        // advancing 16 bf16 along K = 32 bytes = 2 descriptor address units
                        tc::mma_bf16_ss(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                    }
                    tc::mma_commit(&sh->empty[s]);          // frees the stage once these MMAs have read it
                }
                if (ok) tc::mma_commit(&sh->tmem_full);
            }
            if (!ok) {
                if (*abort_flag == 0) report_error(p.status, CTCSD_ERR_TIMEOUT, 2);
                *abort_flag = 1;
            }
        }
    } else {
        // ---------------- epilogue: arg-max of each accumulator row ----------------
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        const int row_in_tile = q * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        int ucount = 0;
        bool ok = true;
        for (int u = u0; u < u1 && ok; ++u, ++ucount) {
            const int nt = u / p.m_tiles, mt = u - nt * p.m_tiles;
            const int n0 = nt * p.Nt;
            const int row = mt * kTileM + row_in_tile;
            if (!tc::mbar_wait(&sh->tmem_full, (uint32_t)ucount & 1u, abort_flag)) { ok = false; break; }
            tc::tc_fence_after_sync();
            float best = -INFINITY;
            int best_idx = 0x7fffffff;
            for (int c0 = 0; c0 < p.Nt; c0 += 32) {
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
                    const float v = __uint_as_float(r[j]);
                    const int col = n0 + c0 + j;
                    if (col < p.V && c0 + j < p.Nt) {
                        if (v > best) { best = v; best_idx = col; }
                        if (p.logits_dbg != nullptr && row < p.M) p.logits_dbg[(size_t)row * p.V + col] = v;
                    }
                }
            }
            tc::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&sh->tmem_empty);
            // fold this tile's winner into the row's global maximum: larger logit first, equal
            // logits -> lower id (the id is stored complemented in the low word)
            if (row < p.M && best_idx != 0x7fffffff) {
                const unsigned u = __float_as_uint(best);
                const unsigned sortable = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
                atomicMax(p.keys + row, ((unsigned long long)sortable << 32) | (0xffffffffu - (unsigned)best_idx));
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
        tc::tmem_dealloc(tmem_base, 256);
    }
    if (tid == 0) {
        unsigned t = atomicAdd(p.counter, 1u);
        sh->is_last = (t == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!sh->is_last) return;
    __threadfence();
    const bool good = sh->abort_flag == 0;
    for (int row = tid; row < p.M; row += kThreads) {
        const unsigned long long key = __ldcg(p.keys + row);
        if (good) p.out_argmax[row] = (int)(0xffffffffu - (unsigned)(key & 0xffffffffull));
        p.keys[row] = 0ull;
    }
    __syncthreads();
    if (good)
        for (int b = warp; b < p.acc.B; b += kThreads / 32) greedy_accept_warp(p.acc, b, lane);
    if (tid == 0) *p.counter = 0u;
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

}  // namespace

bool lm_head_tc_supported(const Handle* h) {
    const ctcsd_config& c = h->cfg;
    return c.dtype == CTCSD_DTYPE_BF16 && c.H % 8 == 0 && c.H >= 64 && c.V >= 16;
}

int launch_lm_head_tc(Handle* h, cudaStream_t stream, int M, const void* hn, const void* Wl,
                      int* out_argmax, float* out_logits_dbg, const AcceptParams& acc) {
    const ctcsd_config& c = h->cfg;
    if (!lm_head_tc_supported(h)) return CTCSD_ERR_UNSUPPORTED;

    TcParams p;
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
    p.n_tiles = (c.V + p.Nt - 1) / p.Nt;
    if (p.m_tiles * kTileM > h->lay.lm_key_count) return CTCSD_ERR_WORKSPACE;
    const int stage_bytes = kABytes + p.Nt * 128;
    int stages = (int)((220 * 1024 - (int)sizeof(TcShared) - 1024) / stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return CTCSD_ERR_UNSUPPORTED;
    p.stages = stages;
    p.keys = reinterpret_cast<unsigned long long*>(h->ws + h->lay.lm_key_off);
    p.acc = acc;
    p.counter = counter_ptr(h) + 1;
    p.out_argmax = out_argmax;
    p.logits_dbg = out_logits_dbg;
    p.status = status_ptr(h);

    CUtensorMap tmA, tmW;
    if (!make_map(&tmA, hn, M, c.H, kTileM)) return CTCSD_ERR_CUDA;
    if (!make_map(&tmW, Wl, c.V, c.H, p.Nt)) return CTCSD_ERR_CUDA;

    const size_t smem = (size_t)stages * stage_bytes + sizeof(TcShared) + 1024;
    CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(lm_head_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    long long units = (long long)p.n_tiles * p.m_tiles;
    int grid = (int)(units < h->num_sms ? units : h->num_sms);
    CTCSD_CUDA_CHECK(h, launch_pdl(lm_head_tc_kernel, dim3(grid), dim3(kThreads), smem, stream, 1, tmA, tmW, p));
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}

}  // namespace ctcsd
