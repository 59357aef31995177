// ctcsd_topk_collapse: slot paths -> CTC collapse -> dedup + alignment-sum score -> top-N.
//
// One CTA per sequence.  The at most T*k <= 64 distinct tokens of the per-slot lists get
// local ids in ascending token order, so a collapsed sequence packs into one 64-bit key
// (length in the top bits, then 6 bits per position) whose unsigned order is exactly
// "shorter first, then token ids lexicographically ascending".  Keys are deduplicated in a
// shared-memory hash table.  Scores are formed in float64; the sum over a candidate's
// alignments is accumulated in 64-bit fixed point relative to the candidate's best
// alignment, which makes it independent of the order in which threads arrive.
#include "common.cuh"

#include <math.h>

namespace ctcsd {
namespace {

constexpr int kMaxThreads = 512;
// threads of the running CTA (the kernels are launched with 512, or with fewer where a sequence has
// little work per slot: a block-wide barrier costs less with fewer warps)
#define NTHR ((int)blockDim.x)
constexpr unsigned long long kEmpty = ~0ull;
constexpr int kBlankMark = 255;
constexpr double kFix = 1125899906842624.0;          // 2^50
constexpr int kBeamCap = 2048;                       // hash capacity for one beam step

struct CollapseParams {
    const int* topk_id;      // [M,T,k]
    const float* topk_lp;    // [M,T,k]
    const int* sel_row;      // [B] or null
    int M, T, k, V, topN, beam, score_mode;
    int npaths;              // k^T (enumeration)
    unsigned k_magic;        // floor(2^32 / k) + 1: x / k == umulhi(x, k_magic) for x < 2^16
    int cap;                 // hash capacity (power of two)
    int* out_cand_tok;       // [B,topN,T]
    int* out_cand_len;       // [B,topN]
    float* out_cand_score;   // [B,topN]
    int* out_n_cand;         // [B]
    int* status;
};

__device__ __forceinline__ int key_len(unsigned long long key) { return (int)(key >> 48); }
__device__ __forceinline__ int key_tok(unsigned long long key, int i) { return (int)((key >> (6 * (7 - i))) & 63ull); }
__device__ __forceinline__ unsigned long long key_append(unsigned long long key, int lid) {
    int len = key_len(key);
    return (key & 0x0000ffffffffffffull) | ((unsigned long long)(len + 1) << 48) |
           ((unsigned long long)lid << (6 * (7 - len)));
}

__device__ __forceinline__ unsigned hash_key(unsigned long long key, int cap) {
    unsigned long long h = key * 0x9E3779B97F4A7C15ull;
    return (unsigned)(h >> 40) & (unsigned)(cap - 1);
}

// Finds or claims the slot of `key`.  The table never fills (capacity >= 2x the entries).
__device__ __forceinline__ int table_insert(unsigned long long* keys, int cap, unsigned long long key,
                                            bool* was_there = nullptr) {
    unsigned s = hash_key(key, cap);
    for (int probe = 0; probe < cap; ++probe) {
        unsigned long long cur = keys[s];
        if (cur == key) { if (was_there) *was_there = true; return (int)s; }
        if (cur == kEmpty) {
            unsigned long long old = atomicCAS(&keys[s], kEmpty, key);
            if (old == kEmpty) return (int)s;
            if (old == key) { if (was_there) *was_there = true; return (int)s; }
        }
        s = (s + 1) & (unsigned)(cap - 1);
    }
    return -1;
}

// Appends to a list whose length is one shared counter: the lanes of a warp that have something
// to append are counted with one ballot and claim their places with ONE atomic (hundreds of
// threads incrementing the same shared word one by one is what a list build otherwise costs).
// Every lane of the warp must call it; returns the place of this lane's item (if `has`).
__device__ __forceinline__ int warp_append(int* counter, bool has) {
    const unsigned m = __ballot_sync(0xffffffffu, has);
    const int lane = threadIdx.x & 31;
    int base = 0;
    if (lane == 0 && m != 0u) base = atomicAdd(counter, __popc(m));
    base = __shfl_sync(0xffffffffu, base, 0);
    return base + __popc(m & ((1u << lane) - 1u));
}

__device__ __forceinline__ long long dbl_sortable(double d) {
    long long v = __double_as_longlong(d);
    return v ^ ((v >> 63) & 0x7fffffffffffffffll);
}
__device__ __forceinline__ double sortable_dbl(long long v) {
    return __longlong_as_double(v ^ ((v >> 63) & 0x7fffffffffffffffll));
}

// (score, key) a precedes b: higher score; equal scores -> smaller key (shorter, then lexicographic)
__device__ __forceinline__ bool precedes(double sa, unsigned long long ka, double sb, unsigned long long kb) {
    return sa > sb || (sa == sb && ka < kb);
}

// Shared bookkeeping common to both modes: the slot lists and the local token ids.
struct SlotLists {
    int tok[CTCSD_MAX_T * CTCSD_MAX_K];        // token id of (t, j)
    double lp[CTCSD_MAX_T * CTCSD_MAX_K];
    unsigned char lid[CTCSD_MAX_T * CTCSD_MAX_K];   // local id, kBlankMark for the blank
    int sorted_tok[64];                        // local id -> token id
};

__device__ void load_slot_lists(const CollapseParams& p, int row, SlotLists& sl) {
    __shared__ unsigned char s_first[CTCSD_MAX_T * CTCSD_MAX_K];
    const int n = p.T * p.k;
    const int tid = threadIdx.x;
    if (tid < n) {
        sl.tok[tid] = p.topk_id[(size_t)row * n + tid];
        sl.lp[tid] = (double)p.topk_lp[(size_t)row * n + tid];
    }
    __syncthreads();
    if (tid < n) {                                   // is (t, j) the first occurrence of its token?
        const int me = sl.tok[tid];
        bool first = me != p.V;
        for (int q = 0; q < tid; ++q) first = first && (sl.tok[q] != me);
        s_first[tid] = first ? 1 : 0;
    }
    __syncthreads();
    if (tid < n) {
        const int me = sl.tok[tid];
        if (me == p.V) {
            sl.lid[tid] = kBlankMark;
        } else {
            int cnt = 0;                             // local id = number of distinct smaller tokens
            for (int j = 0; j < n; ++j) cnt += (s_first[j] && sl.tok[j] < me) ? 1 : 0;
            sl.lid[tid] = (unsigned char)cnt;
            if (s_first[tid]) sl.sorted_tok[cnt] = me;
        }
    }
    __syncthreads();
}

// Block-wide bitonic sort of n2 (a power of two) entries into "best first" order:
// higher score first, equal scores -> smaller key.  ix is an optional payload.
__device__ void bitonic_sort_best_first(double* sc, unsigned long long* ky, int* ix, int n2) {
    const int tid = threadIdx.x;
    for (int k = 2; k <= n2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = tid; t < (n2 >> 1); t += NTHR) {
                const int lo = t & (j - 1);
                const int i = ((t - lo) << 1) | lo;
                const int q = i | j;
                const bool up = (i & k) == 0;
                const double si = sc[i], sq = sc[q];
                const unsigned long long ki = ky[i], kq = ky[q];
                const bool swap = up ? precedes(sq, kq, si, ki) : precedes(si, ki, sq, kq);
                if (swap) {
                    sc[i] = sq; sc[q] = si;
                    ky[i] = kq; ky[q] = ki;
                    if (ix) { int a = ix[i]; ix[i] = ix[q]; ix[q] = a; }
                }
            }
            __syncthreads();
        }
    }
}

constexpr int kSelMax = 256;     // most near-threshold entries the exact tie-break handles
constexpr int kRankMax = 32;     // the radix rounds go on until this few are left (one comparison round per entry)

struct SelectScratch {
    unsigned hist[2][256];         // one per round parity; all zero between calls
    int win[CTCSD_MAX_BEAM + 8];   // indices of selected entries (unordered)
    int cand[kSelMax];             // indices of entries on the threshold
    unsigned fmax, fmin;           // range of the images (RANGE_GIVEN: accumulated by the caller)
    unsigned thr[2];               // per round parity: what the scanning warp found
    int need[2], ncand[2];
    int nwin, ccnt;                // list lengths; zero between calls
};

__device__ __forceinline__ void select_scratch_init(SelectScratch& S) {
    for (int i = threadIdx.x; i < 512; i += NTHR) (&S.hist[0][0])[i] = 0u;
    if (threadIdx.x == 0) { S.fmax = 0u; S.fmin = 0xffffffffu; S.nwin = 0; S.ccnt = 0; }
}

// float32 image of a score as an unsigned integer whose order matches the score's
__device__ __forceinline__ unsigned sortable_f32(double v) {
    unsigned u = __float_as_uint((float)v);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
// 32-bit image used by the radix select.  MASS = false: the score is a logarithm (any sign), its
// float32 value is used.  MASS = true: the score is a non-negative probability mass that may be
// far below the float32 range; the upper word of the float64 (exponent and 20 mantissa bits) is
// monotone for non-negative values.
template <bool MASS> __device__ __forceinline__ unsigned select_image(double v) {
    if constexpr (MASS) return (unsigned)__double2hiint(v);
    else return sortable_f32(v);
}

__device__ __forceinline__ int next_pow2(int v) {
    int n = 2;
    while (n < v) n <<= 1;
    return n;
}

// Selects the `need` (<= CTCSD_MAX_BEAM) best of `count` entries and writes their indices,
// best first (in any order when `ordered` is false), to sel[]; returns how many were selected.
// A radix select on a 32-bit image of the scores finds the threshold in O(count) work per round of
// eight bits (the bits all images share are skipped); once at most kRankMax entries sit on the
// threshold they are ranked exactly (float64 score, then key).  If more than kSelMax entries
// still sit there at full image resolution the arrays (padded to a power of two, capacity >=
// next_pow2(count)) are sorted in place instead and sel[] becomes the identity.
// RANGE_GIVEN: the caller has run select_scratch_init once, and accumulates the largest and the
// smallest image of this call's entries in S.fmax / S.fmin (and resets them afterwards); this
// saves the pass that finds them.  Otherwise the call is self-contained.
// A round costs two barriers: histograms and the scanning warp's results alternate between two
// copies, so nobody has to wait before the next round overwrites them.
template <bool MASS = false, bool RANGE_GIVEN = false>
__device__ int block_select_top(double* sc, unsigned long long* ky, int* ix, int count, int need, int* sel,
                                SelectScratch& S, bool ordered = true, int* status = nullptr) {
    const int tid = threadIdx.x, lane = tid & 31;
    if (need > count) need = count;
    if constexpr (!RANGE_GIVEN) {
        select_scratch_init(S);
        __syncthreads();
    }
    int* win = ordered ? S.win : sel;                  // an unordered selection goes straight to the caller
    if (count > need) {
        if constexpr (!RANGE_GIVEN) {
            unsigned lmax = 0u, lmin = 0xffffffffu;
            for (int i = tid; i < count; i += NTHR) {
                const unsigned f = select_image<MASS>(sc[i]);
                lmax = max(lmax, f);
                lmin = min(lmin, f);
            }
            lmax = __reduce_max_sync(0xffffffffu, lmax);
            lmin = __reduce_min_sync(0xffffffffu, lmin);
            if (lane == 0) { atomicMax(&S.fmax, lmax); atomicMin(&S.fmin, lmin); }
            __syncthreads();
        }
        const unsigned diff = S.fmax ^ S.fmin;
        // bits at and above `lo` agree for all entries; walk down 8 bits at a time
        int lo = diff ? (31 - __clz(diff)) + 1 : 0;
        unsigned thr = lo < 32 ? (S.fmax >> lo) : 0u;
        int remaining = need;
        int ncand = count;
        for (int round = 0; lo > 0 && ncand > remaining; ++round) {
            const int nlo = lo > 8 ? lo - 8 : 0;
            const int width = lo - nlo;
            unsigned* H = S.hist[round & 1];
            for (int i = tid; i < count; i += NTHR) {
                const unsigned f = select_image<MASS>(sc[i]);
                const unsigned top = lo < 32 ? (f >> lo) : 0u;
                if (top == thr) atomicAdd(&H[(f >> nlo) & ((1u << width) - 1u)], 1u);
            }
            __syncthreads();
            if (tid < 32) {
                // lane owns digits [8*lane, 8*lane+8); find the digit where the count from the top reaches `remaining`
                unsigned h[8], mine = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) { h[q] = H[8 * lane + q]; H[8 * lane + q] = 0u; mine += h[q]; }
                unsigned suf = mine;                      // suffix sum: entries in this lane and above
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    unsigned v = __shfl_down_sync(0xffffffffu, suf, o);
                    if (lane + o < 32) suf += v;
                }
                const unsigned above = suf - mine;
                if (above < (unsigned)remaining && above + mine >= (unsigned)remaining) {
                    unsigned acc = above;
#pragma unroll
                    for (int q = 7; q >= 0; --q) {
                        if (acc < (unsigned)remaining && acc + h[q] >= (unsigned)remaining) {
                            S.thr[round & 1] = (thr << width) | (unsigned)(8 * lane + q);
                            S.need[round & 1] = remaining - (int)acc;
                            S.ncand[round & 1] = (int)h[q];
                        }
                        acc += h[q];
                    }
                }
            }
            __syncthreads();
            thr = S.thr[round & 1]; remaining = S.need[round & 1]; ncand = S.ncand[round & 1];
            lo = nlo;
            if (ncand <= kRankMax) break;
        }
        if (ncand > remaining && ncand > kSelMax) {
            // too many entries share the threshold even at full image resolution: sort everything
            const int n2 = next_pow2(count);
            for (int i = count + tid; i < n2; i += NTHR) { sc[i] = MASS ? -1.0 : -INFINITY; ky[i] = kEmpty; if (ix) ix[i] = 0; }
            __syncthreads();
            bitonic_sort_best_first(sc, ky, ix, n2);
            for (int r = tid; r < need; r += NTHR) sel[r] = r;
            __syncthreads();
            return need;
        }
        // gather definite winners (above the threshold) and the entries on it
        for (int i0 = 0; i0 < count; i0 += NTHR) {          // the same trip count for every thread
            const int i = i0 + tid;
            bool is_win = false, is_cand = false;
            if (i < count) {
                const unsigned f = select_image<MASS>(sc[i]);
                const unsigned top = lo < 32 ? (f >> lo) : 0u;
                is_win = top > thr;
                is_cand = top == thr;
            }
            const int aw = warp_append(&S.nwin, is_win);
            const int ac = warp_append(&S.ccnt, is_cand);
            if (is_win && CTCSD_IN_BOUNDS(status, 5, aw, CTCSD_MAX_BEAM + 8)) win[aw] = i;
            if (is_cand && CTCSD_IN_BOUNDS(status, 6, ac, kSelMax)) S.cand[ac] = i;
        }
        __syncthreads();
        // exact ranking among the threshold entries: one warp per entry, its lanes share the
        // comparisons (a rank is the number of entries that precede it)
        for (int c = tid >> 5; c < ncand; c += NTHR / 32) {
            const int i = S.cand[c];
            const double si = sc[i];
            const unsigned long long ki = ky[i];
            int rank = 0;
            for (int d = lane; d < ncand; d += 32) {
                const int j = S.cand[d];
                rank += precedes(sc[j], ky[j], si, ki) ? 1 : 0;
            }
            rank = __reduce_add_sync(0xffffffffu, rank);
            if (lane == 0 && rank < remaining) win[atomicAdd(&S.nwin, 1)] = i;
        }
        __syncthreads();
        if (tid == 0) { S.nwin = 0; S.ccnt = 0; }      // (next read after the caller's barrier or this call's last one)
    } else {
        for (int i = tid; i < count; i += NTHR) win[i] = i;
        __syncthreads();
    }
    if (!ordered) return need;                        // the caller only needs the set
    // order the winners, again one warp per winner
    for (int w = tid >> 5; w < need; w += NTHR / 32) {
        const int i = S.win[w];
        const double si = sc[i];
        const unsigned long long ki = ky[i];
        int rank = 0;
        for (int d = lane; d < need; d += 32) {
            const int j = S.win[d];
            rank += precedes(sc[j], ky[j], si, ki) ? 1 : 0;
        }
        rank = __reduce_add_sync(0xffffffffu, rank);
        if (lane == 0) sel[rank] = i;
    }
    __syncthreads();
    return need;
}

// Writes the candidates: the selected entries in ranked order, the empty sequence skipped.
// `total_nonempty` is the number of distinct non-empty sequences that exist.
__device__ void emit_candidates(const CollapseParams& p, int b, const SlotLists& sl, const double* sc,
                                const unsigned long long* ky, const int* sel, int nsel, int total_nonempty) {
    __shared__ int s_empty_at;
    const int tid = threadIdx.x;
    if (tid == 0) s_empty_at = 0x7fffffff;
    int* ctok = p.out_cand_tok + (size_t)b * p.topN * p.T;
    int* clen = p.out_cand_len + (size_t)b * p.topN;
    float* cscore = p.out_cand_score + (size_t)b * p.topN;
    for (int i = tid; i < p.topN * p.T; i += NTHR) ctok[i] = -1;
    for (int i = tid; i < p.topN; i += NTHR) { clen[i] = 0; cscore[i] = -INFINITY; }
    __syncthreads();
    for (int e = tid; e < nsel; e += NTHR)
        if (key_len(ky[sel[e]]) == 0) s_empty_at = e;
    __syncthreads();
    const int empty_at = s_empty_at;
    for (int e = tid; e < nsel; e += NTHR) {
        if (e == empty_at) continue;
        const int rank = e - (empty_at < e ? 1 : 0);
        if (rank >= p.topN) continue;
        const unsigned long long key = ky[sel[e]];
        const int len = key_len(key);
        if (!CTCSD_IN_BOUNDS(p.status, 1, rank, p.topN) || !CTCSD_IN_BOUNDS(p.status, 2, len, p.T + 1)) continue;
        clen[rank] = len;
        cscore[rank] = (float)sc[sel[e]];
        for (int l = 0; l < len; ++l) ctok[rank * p.T + l] = sl.sorted_tok[key_tok(key, l)];
    }
    if (tid == 0) {
        const int nonempty = total_nonempty >= 0 ? total_nonempty : nsel - (empty_at != 0x7fffffff ? 1 : 0);
        p.out_n_cand[b] = nonempty < p.topN ? nonempty : p.topN;
    }
}

// Decodes path index -> per-slot choices (last slot fastest), returning the collapsed
// sequence's key and the path's log-probability (summed in slot order).
__device__ __forceinline__ unsigned long long path_key_and_score(const CollapseParams& p, const SlotLists& sl,
                                                                 int path, double& score) {
    unsigned rem = (unsigned)path;
    int digit[CTCSD_MAX_T];
#pragma unroll
    for (int t = CTCSD_MAX_T - 1; t >= 0; --t) {
        if (t < p.T) {
            const unsigned q = __umulhi(rem, p.k_magic);     // rem / k for rem < 2^16, k <= 8
            digit[t] = (int)(rem - q * (unsigned)p.k);
            rem = q;
        } else {
            digit[t] = 0;
        }
    }
    double s = 0.0;
    unsigned long long key = 0ull;
    int prev = -1;
#pragma unroll
    for (int t = 0; t < CTCSD_MAX_T; ++t) {
        if (t < p.T) {
            const int e = t * p.k + digit[t];
            s += sl.lp[e];
            const int m = sl.lid[e];
            if (m != prev && m != kBlankMark) key = key_append(key, m);
            prev = m;
        }
    }
    score = s;
    return key;
}

// ---------------------------------------------------------------------------------------
// Exhaustive enumeration of the k^T slot paths
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kMaxThreads, 1) collapse_enum_kernel(CollapseParams p) {
    extern __shared__ __align__(16) unsigned char dyn[];
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(dyn);             // [cap]
    long long* best = reinterpret_cast<long long*>(keys + p.cap);                      // [cap] sortable max, then score
    unsigned long long* fsum = reinterpret_cast<unsigned long long*>(best + p.cap);    // [cap] fixed-point sum
    unsigned short* path_slot = reinterpret_cast<unsigned short*>(fsum + p.cap);       // [npaths]
    __shared__ SlotLists sl;
    __shared__ SelectScratch S;
    __shared__ int s_sel[CTCSD_MAX_BEAM + 8];
    __shared__ int s_count, s_has_empty, s_merged;

    const int b = blockIdx.x, tid = threadIdx.x;
    pdl_wait();                      // the per-slot lists come from the preceding kernel
    pdl_trigger();
    const int row = p.sel_row ? p.sel_row[b] : b;
    if (row < 0 || row >= p.M) {
        if (tid == 0) { report_error(p.status, CTCSD_ERR_INVALID_ARG, b); p.out_n_cand[b] = 0; }
        return;
    }
    load_slot_lists(p, row, sl);
    const long long neg_inf_sortable = dbl_sortable(-INFINITY);
    for (int i = tid; i < p.cap; i += NTHR) { keys[i] = kEmpty; best[i] = neg_inf_sortable; fsum[i] = 0ull; }
    if (tid == 0) { s_count = 0; s_has_empty = 0; s_merged = 0; }
    __syncthreads();

    // pass 1: collapse every path, claim a table slot, track the best alignment
    for (int path = tid; path < p.npaths; path += NTHR) {
        double s;
        const unsigned long long key = path_key_and_score(p, sl, path, s);
        bool was_there = false;
        int slot = table_insert(keys, p.cap, key, &was_there);
        if (was_there) s_merged = 1;                     // some candidate has more than one alignment
        if (slot < 0) { report_error(p.status, CTCSD_ERR_INTERNAL, 1); slot = 0; }
        path_slot[path] = (unsigned short)slot;
        atomicMax(&best[slot], dbl_sortable(s));
    }
    __syncthreads();

    // pass 2: sum exp(s - best) per candidate in fixed point (order independent).  The best
    // alignment itself contributes exp(0) = 1 exactly, so it needs no call to exp.  When no two
    // paths collapsed to the same sequence every sum is that single 1 and the pass is skipped.
    const bool sums = p.score_mode == CTCSD_SCORE_SUM && s_merged != 0;
    if (sums) {
        for (int path = tid; path < p.npaths; path += NTHR) {
            double s;
            path_key_and_score(p, sl, path, s);
            const int slot = path_slot[path];
            const long long bs = best[slot];
            unsigned long long term = 1ull << 50;
            if (dbl_sortable(s) != bs) term = __double2ull_rn(exp(s - sortable_dbl(bs)) * kFix);
            atomicAdd(&fsum[slot], term);
        }
    }
    __syncthreads();
    double* score = reinterpret_cast<double*>(best);
    for (int i = tid; i < p.cap; i += NTHR) {
        if (keys[i] == kEmpty) continue;
        const double mx = sortable_dbl(best[i]);
        double sc = mx;
        // a single alignment sums to exactly 1: log(1) = 0
        if (sums && fsum[i] != (1ull << 50)) sc = mx + log((double)fsum[i] * (1.0 / kFix));
        score[i] = sc;
    }
    __syncthreads();

    // compact the distinct candidates into the (now free) sum array, pick the best topN (+1
    // because the empty sequence may be among them) and write them out
    double* c_sc = reinterpret_cast<double*>(fsum);                     // [cap/2]
    unsigned long long* c_ky = fsum + (p.cap >> 1);                     // [cap/2]
    for (int i0 = 0; i0 < p.cap; i0 += NTHR) {
        const int i = i0 + tid;
        const unsigned long long ki = i < p.cap ? keys[i] : kEmpty;
        const bool has = ki != kEmpty;
        const double si = has ? score[i] : 0.0;
        const int at = warp_append(&s_count, has);
        if (!has || !CTCSD_IN_BOUNDS(p.status, 4, at, p.cap >> 1)) continue;
        if (ki == 0ull) s_has_empty = 1;
        c_sc[at] = si;
        c_ky[at] = ki;
    }
    __syncthreads();
    const int count = s_count;
    const int nsel = block_select_top(c_sc, c_ky, nullptr, count, p.topN + 1, s_sel, S, true, p.status);
    emit_candidates(p, b, sl, c_sc, c_ky, s_sel, nsel, count - s_has_empty);
}

// ---------------------------------------------------------------------------------------
// CTC prefix beam search over the per-slot lists
// ---------------------------------------------------------------------------------------
// Finds `key` in a set built with table_insert; returns its payload index or -1.
__device__ __forceinline__ int set_lookup(const unsigned long long* keys, const short* val, int cap, unsigned long long key) {
    unsigned s = hash_key(key, cap);
    for (int probe = 0; probe < cap; ++probe) {
        const unsigned long long cur = keys[s];
        if (cur == key) return val[s];
        if (cur == kEmpty) return -1;
        s = (s + 1) & (unsigned)(cap - 1);
    }
    return -1;
}

// What one slot makes of the beam.  A prefix e with masses (pb: alignments ending in the blank, pnb:
// ending in its last token) and a slot with symbols m_j of probability p_j give
//   e itself   pb'  = (pb + pnb) p_blank          (if the blank is among the slot's symbols)
//              pnb' = pnb p_last(e)               (if e's last token is)
//   e + m      pnb' = (m == last(e) ? pb : pb + pnb) p_m      for every non-blank m.
// Two different (e, m) never give the same sequence, and two prefixes of the beam are different
// sequences, so the only merging there is happens when e + m is itself a prefix e' of the beam:
// the extension's mass then joins pnb' of e'.  Hence no hash table of candidates: the beam's own
// keys go into a small set (one insert per prefix), every extension looks itself up there (a
// read-only probe); a hit hands its mass to the beam prefix through a one-writer inbox, a miss is
// a new candidate whose mass is final and goes straight onto the selection list.  The prefixes
// themselves follow once the inboxes are complete.
__global__ void __launch_bounds__(kMaxThreads, 1) collapse_beam_kernel(CollapseParams p) {
    extern __shared__ __align__(16) unsigned char dyn[];
    const int cap = p.cap;                   // candidates per slot rounded up to a power of two (the fallback sort needs it)
    double* c_sc = reinterpret_cast<double*>(dyn);                            // [cap] masses of the candidates
    unsigned long long* c_ky = reinterpret_cast<unsigned long long*>(c_sc + cap);
    int* c_ix = reinterpret_cast<int*>(c_ky + cap);                           // [cap] beam index of a prefix that stayed, -1 for a new one
    __shared__ unsigned long long h_key[4 * CTCSD_MAX_BEAM];                  // the beam's keys as a set (load <= 1/4)
    __shared__ short h_val[4 * CTCSD_MAX_BEAM];
    __shared__ double ext_in[CTCSD_MAX_BEAM];                                 // mass an extension hands to a beam prefix
    __shared__ double st_pb[CTCSD_MAX_BEAM], st_pnb[CTCSD_MAX_BEAM];          // the new masses of a prefix that stays
    __shared__ unsigned long long bm_key[CTCSD_MAX_BEAM];
    __shared__ double bm_pb[CTCSD_MAX_BEAM], bm_pnb[CTCSD_MAX_BEAM], bm_tot[CTCSD_MAX_BEAM];
    __shared__ int s_nbeam, s_next;
    __shared__ SlotLists sl;
    __shared__ SelectScratch S;
    __shared__ int s_sel[CTCSD_MAX_BEAM + 8];

    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    pdl_wait();                      // the per-slot lists come from the preceding kernel
    pdl_trigger();
    const int row = p.sel_row ? p.sel_row[b] : b;
    if (row < 0 || row >= p.M) {
        if (tid == 0) { report_error(p.status, CTCSD_ERR_INVALID_ARG, b); p.out_n_cand[b] = 0; }
        return;
    }
    load_slot_lists(p, row, sl);
    // The search runs on probability masses, not on their logarithms: a prefix's mass is a sum of
    // products, which in the log domain costs an exp and a log1p in float64 per addition.  Every
    // slot's probabilities are taken relative to the slot's best symbol (so the best path has mass
    // 1 and nothing overflows; a path more than ~700 nats below the best one underflows to "no
    // alignment"); the logarithm of the common factor is added back when the scores are written.
    __shared__ double s_pr[CTCSD_MAX_T * CTCSD_MAX_K];
    __shared__ double s_logoff;
    int hcap = 4;                                        // set capacity: a power of two >= 4 * beam
    while (hcap < 4 * p.beam) hcap <<= 1;
    if (tid < p.T * p.k) {
        const int t = tid / p.k;
        double mx = sl.lp[t * p.k];
        for (int j = 1; j < p.k; ++j) mx = fmax(mx, sl.lp[t * p.k + j]);
        s_pr[tid] = exp(sl.lp[tid] - mx);
        if (tid == 0) {
            double off = 0.0;
            for (int q = 0; q < p.T; ++q) {
                double m2 = sl.lp[q * p.k];
                for (int j = 1; j < p.k; ++j) m2 = fmax(m2, sl.lp[q * p.k + j]);
                off += m2;
            }
            s_logoff = off;
        }
    }
    select_scratch_init(S);
    for (int i = tid; i < hcap; i += NTHR) h_key[i] = kEmpty;
    for (int i = tid; i < p.beam; i += NTHR) ext_in[i] = 0.0;
    if (tid == 0) { bm_key[0] = 0ull; bm_pb[0] = 1.0; bm_pnb[0] = 0.0; bm_tot[0] = 1.0; s_nbeam = 1; s_next = 0; }
    __syncthreads();
    if (tid == 0) { const int at = table_insert(h_key, hcap, 0ull); if (at >= 0) h_val[at] = 0; }
    __syncthreads();

    for (int t = 0; t < p.T; ++t) {
        const int nbeam = s_nbeam;
        const int next = nbeam * p.k;                    // extensions: item e * k + j
        const int nitem = next + nbeam;                  // then the prefixes themselves
        unsigned lmax = 0u, lmin = 0xffffffffu;          // range of the candidates' images, for the selection
        // ---- extensions look themselves up in the beam; the prefixes work out what stays with them ----
        for (int w0 = 0; w0 < nitem; w0 += NTHR) {       // (whole warps go round: the list append is a warp operation)
            const int w = w0 + tid;
            bool has = false;
            unsigned long long ck = kEmpty;
            double val = 0.0;
            if (w < next) {
                const int e = w / p.k, j = w - e * p.k;
                const int m = sl.lid[t * p.k + j];
                if (m != kBlankMark) {
                    const unsigned long long key = bm_key[e];
                    const int len = key_len(key);
                    const int last = len > 0 ? key_tok(key, len - 1) : -1;
                    val = (m == last ? bm_pb[e] : bm_tot[e]) * s_pr[t * p.k + j];
                    if (val != 0.0) {                    // (a symbol or a prefix of mass zero reaches nothing)
                        ck = key_append(key, m);
                        const int hit = set_lookup(h_key, h_val, hcap, ck);
                        if (hit >= 0) ext_in[hit] = val; // e + m is beam prefix `hit`, and this its only such donor
                        else has = true;
                    }
                }
            } else if (w < nitem) {
                const int e = w - next;
                const unsigned long long key = bm_key[e];
                const int len = key_len(key);
                const int last = len > 0 ? key_tok(key, len - 1) : -1;
                const double pnb = bm_pnb[e], tot = bm_tot[e];
                double cpb = 0.0, cpnb = 0.0;
                for (int q = 0; q < p.k; ++q) {
                    const int m = sl.lid[t * p.k + q];
                    const double pr = s_pr[t * p.k + q];
                    if (m == kBlankMark) cpb = tot * pr;
                    else if (m == last) cpnb = pnb * pr;
                }
                st_pb[e] = cpb;
                st_pnb[e] = cpnb;
            }
            const int at = warp_append(&s_next, has);
            if (!has || !CTCSD_IN_BOUNDS(p.status, 3, at, cap)) continue;
            c_sc[at] = val;
            c_ky[at] = ck;
            c_ix[at] = -1;
            const unsigned f = select_image<true>(val);
            lmax = max(lmax, f);
            lmin = min(lmin, f);
        }
        __syncthreads();
        // ---- the prefixes collect what extensions handed them and join the list ----
        for (int e0 = 0; e0 < nbeam; e0 += NTHR) {
            const int e = e0 + tid;
            double tot = 0.0;
            if (e < nbeam) {
                const double pnb = st_pnb[e] + ext_in[e];
                ext_in[e] = 0.0;
                st_pnb[e] = pnb;
                tot = st_pb[e] + pnb;
            }
            const bool has = tot != 0.0;                 // (a mass that underflowed has no alignment left)
            const int at = warp_append(&s_next, has);
            if (!has || !CTCSD_IN_BOUNDS(p.status, 4, at, cap)) continue;
            c_sc[at] = tot;
            c_ky[at] = bm_key[e];
            c_ix[at] = e;
            const unsigned f = select_image<true>(tot);
            lmax = max(lmax, f);
            lmin = min(lmin, f);
        }
        for (int i = tid; i < hcap; i += NTHR) h_key[i] = kEmpty;       // every lookup is done
        lmax = __reduce_max_sync(0xffffffffu, lmax);
        lmin = __reduce_min_sync(0xffffffffu, lmin);
        if (lane == 0 && lmax >= lmin) { atomicMax(&S.fmax, lmax); atomicMin(&S.fmin, lmin); }
        __syncthreads();
        const int count = s_next;
        // ---- the `beam` heaviest: between slots a set; only the last slot's beam is ranked ----
        const int keep = block_select_top<true, true>(c_sc, c_ky, c_ix, count, p.beam, s_sel, S, t == p.T - 1, p.status);
        // ---- they become the beam, and its key set ----
        for (int r = tid; r < keep; r += NTHR) {
            const int i = s_sel[r];
            const int e = c_ix[i];
            const unsigned long long ck = c_ky[i];
            const double tot = c_sc[i];
            bm_key[r] = ck;
            bm_pb[r] = e >= 0 ? st_pb[e] : 0.0;
            bm_pnb[r] = e >= 0 ? st_pnb[e] : tot;
            bm_tot[r] = tot;
            const int at = table_insert(h_key, hcap, ck);
            if (at >= 0) h_val[at] = (short)r;
        }
        if (tid == 0) { s_nbeam = keep; s_next = 0; S.fmax = 0u; S.fmin = 0xffffffffu; }
        __syncthreads();
    }
    // the beam is already ranked best first by total mass; scores go out as logarithms
    const int nbeam = s_nbeam;
    for (int r = tid; r < nbeam; r += NTHR) {
        s_sel[r] = r;
        bm_tot[r] = log(bm_tot[r]) + s_logoff;
    }
    __syncthreads();
    emit_candidates(p, b, sl, bm_tot, bm_key, s_sel, nbeam, -1);
}

// ---------------------------------------------------------------------------------------
// Raw-path selection (Sec. 3.3, the paper's own verification layout): the topN most probable
// slot paths, blanks and repeats left in place.  Path probability = product over the slots
// (Eq. 6), summed in slot order in float64; equal scores go to the lower path index (slot 1
// most significant, per-slot rank as the digit).
// ---------------------------------------------------------------------------------------
struct RawParams {
    CollapseParams c;
    int* out_raw_tok;        // [B,topN,T]
    float* out_raw_score;    // [B,topN]
    int* out_n_raw;          // [B]
};

__global__ void __launch_bounds__(kMaxThreads, 1) raw_paths_kernel(RawParams rp) {
    extern __shared__ __align__(16) unsigned char dyn[];
    const CollapseParams& p = rp.c;
    double* sc = reinterpret_cast<double*>(dyn);                                   // [cap]
    unsigned long long* ky = reinterpret_cast<unsigned long long*>(sc + p.cap);    // [cap]
    __shared__ SlotLists sl;
    __shared__ SelectScratch S;
    __shared__ int s_sel[CTCSD_MAX_BEAM + 8];

    const int b = blockIdx.x, tid = threadIdx.x;
    pdl_wait();                      // the per-slot lists come from the preceding kernel
    pdl_trigger();
    const int row = p.sel_row ? p.sel_row[b] : b;
    int* rtok = rp.out_raw_tok + (size_t)b * p.topN * p.T;
    float* rscore = rp.out_raw_score + (size_t)b * p.topN;
    if (row < 0 || row >= p.M) {
        if (tid == 0) { report_error(p.status, CTCSD_ERR_INVALID_ARG, b); rp.out_n_raw[b] = 0; }
        return;
    }
    load_slot_lists(p, row, sl);
    for (int path = tid; path < p.npaths; path += NTHR) {
        double s;
        path_key_and_score(p, sl, path, s);
        sc[path] = s;
        ky[path] = (unsigned long long)path;
    }
    for (int i = tid; i < p.topN * p.T; i += NTHR) rtok[i] = -1;
    for (int i = tid; i < p.topN; i += NTHR) rscore[i] = -INFINITY;
    __syncthreads();
    const int nsel = block_select_top(sc, ky, nullptr, p.npaths, p.topN, s_sel, S, true, p.status);
    for (int e = tid; e < nsel; e += NTHR) {
        const int at = s_sel[e];
        unsigned rem = (unsigned)ky[at];
        rscore[e] = (float)sc[at];
        for (int t = p.T - 1; t >= 0; --t) {
            const unsigned q = rem / (unsigned)p.k;
            rtok[e * p.T + t] = sl.tok[t * p.k + (int)(rem - q * (unsigned)p.k)];
            rem = q;
        }
    }
    if (tid == 0) rp.out_n_raw[b] = nsel;
}

}  // namespace
}  // namespace ctcsd

using namespace ctcsd;

static int next_pow2_host(int v) {
    int n = 2;
    while (n < v) n <<= 1;
    return n;
}

extern "C" int ctcsd_topk_collapse(ctcsd_handle* hh, void* stream, int M, const int* topk_id, const float* topk_lp,
                                   const int* sel_row,
                                   int* out_cand_tok, int* out_cand_len, float* out_cand_score, int* out_n_cand) {
    if (!hh || !topk_id || !topk_lp || !out_cand_tok || !out_cand_len || !out_cand_score || !out_n_cand)
        return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    const ctcsd_config& c = h->cfg;
    if (M < 1) return CTCSD_ERR_INVALID_ARG;
    if (!sel_row && M < c.B) return CTCSD_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    CollapseParams p;
    p.topk_id = topk_id;
    p.topk_lp = topk_lp;
    p.sel_row = sel_row;
    p.M = M; p.T = c.T; p.k = c.k; p.V = c.V; p.topN = c.topN; p.beam = c.beam; p.score_mode = c.score_mode;
    p.npaths = 0; p.cap = 0;
    p.k_magic = (unsigned)((1ull << 32) / (unsigned)c.k) + 1u;
    p.out_cand_tok = out_cand_tok;
    p.out_cand_len = out_cand_len;
    p.out_cand_score = out_cand_score;
    p.out_n_cand = out_n_cand;
    p.status = status_ptr(h);

    if (c.beam > 0) {
        int cap = 64;                            // candidates of one slot: beam * (k + 1), as a power of two
        while (cap < c.beam * (c.k + 1)) cap <<= 1;
        if (cap > kBeamCap) cap = kBeamCap;
        p.cap = cap;
        // (fewer threads per sequence were measured slower at every beam: 128 / 256 / 320 / 512 threads
        // took 96 / 64 / 56 / 52 us at beam 128 and 38 / 28 / 28 / 26 us at beam 64)
        const int beam_threads = kMaxThreads;
        const size_t smem = (size_t)cap * 20;
        CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(collapse_beam_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        CTCSD_CUDA_CHECK(h, launch_pdl(collapse_beam_kernel, dim3(c.B), dim3(beam_threads), smem, s, 1, p));
        CTCSD_LAUNCH_CHECK(h);
        return CTCSD_OK;
    }
    int npaths = 1;
    for (int t = 0; t < c.T; ++t) npaths *= c.k;
    int cap = 64;
    while (cap < 2 * npaths) cap <<= 1;
    p.npaths = npaths;
    p.cap = cap;
    size_t smem = (size_t)cap * 24 + (size_t)npaths * 2;
    if (smem > 48 * 1024)
        CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(collapse_enum_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    CTCSD_CUDA_CHECK(h, launch_pdl(collapse_enum_kernel, dim3(c.B), dim3(kMaxThreads), smem, s, 1, p));
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}

extern "C" int ctcsd_select_raw_paths(ctcsd_handle* hh, void* stream, int M, const int* topk_id, const float* topk_lp,
                                      const int* sel_row, int* out_raw_tok, float* out_raw_score, int* out_n_raw) {
    if (!hh || !topk_id || !topk_lp || !out_raw_tok || !out_raw_score || !out_n_raw) return CTCSD_ERR_INVALID_ARG;
    Handle* h = &hh->h;
    const ctcsd_config& c = h->cfg;
    if (M < 1) return CTCSD_ERR_INVALID_ARG;
    if (!sel_row && M < c.B) return CTCSD_ERR_INVALID_ARG;
    long long npaths = 1;
    for (int t = 0; t < c.T; ++t) {
        npaths *= c.k;
        if (npaths > CTCSD_MAX_PATHS) return CTCSD_ERR_UNSUPPORTED;
    }
    RawParams rp;
    CollapseParams& p = rp.c;
    p.topk_id = topk_id;
    p.topk_lp = topk_lp;
    p.sel_row = sel_row;
    p.M = M; p.T = c.T; p.k = c.k; p.V = c.V; p.topN = c.topN; p.beam = 0; p.score_mode = CTCSD_SCORE_MAX;
    p.npaths = (int)npaths;
    p.cap = next_pow2_host((int)npaths);
    p.k_magic = (unsigned)((1ull << 32) / (unsigned)c.k) + 1u;
    p.out_cand_tok = nullptr; p.out_cand_len = nullptr; p.out_cand_score = nullptr; p.out_n_cand = nullptr;
    p.status = status_ptr(h);
    rp.out_raw_tok = out_raw_tok; rp.out_raw_score = out_raw_score; rp.out_n_raw = out_n_raw;
    const size_t smem = (size_t)p.cap * 16;
    if (smem > 48 * 1024)
        CTCSD_CUDA_CHECK(h, cudaFuncSetAttribute(raw_paths_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    CTCSD_CUDA_CHECK(h, launch_pdl(raw_paths_kernel, dim3(c.B), dim3(kMaxThreads), smem, static_cast<cudaStream_t>(stream), 1, rp));
    CTCSD_LAUNCH_CHECK(h);
    return CTCSD_OK;
}
