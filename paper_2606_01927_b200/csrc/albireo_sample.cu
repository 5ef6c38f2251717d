// Batched token sampler for B200 (sm_100a): kernels and C ABI.
//
// One CTA samples one row of the [B, V] logits matrix (rows are independent, paper
// section 6.1).  Every step of the per-row computation declared in albireo_sample.h runs
// in this file; there is no host-side arithmetic and no fallback.
//
// Two device paths produce the same result:
//   * general path  -- multi-pass radix selection over the whole row (any parameter mix,
//                      any kept-set size); the row is re-read from L2 between passes.
//   * candidate path -- one streaming pass that keeps only the few elements that can
//                      still be among the kept set (rows with a small top-k or a
//                      selective min-p); falls back to the general path when its
//                      on-chip buffers would overflow.
//
// Total order used everywhere: composite C(t) = (key(z_t) << 32) | ~t, where key() is
// the order-preserving map of fp32 bit patterns.  Larger C comes first; all C distinct.
// A kept set is always a prefix of that order, i.e. { t : C(t) >= threshold }.

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>
#include <new>

#include "albireo_sample.h"

namespace {

typedef unsigned long long u64;

constexpr int NT = 512;                 // threads per CTA
constexpr int NWARPS = NT / 32;
constexpr int HIST_BINS = 2048;         // 11-bit digits
constexpr int CNT_CAP = 4096;           // on-chip slots for distinct history ids per row
constexpr int CAND_CAP = 2048;          // candidate buffer entries (candidate path)
constexpr int SORT_MAX = 512;           // most candidates the final stage sorts (== NT)
constexpr int KA_MAX = 256;             // largest top-k the candidate path takes
constexpr int TILE_VECS = 4;            // 16-byte vectors per thread per tile
constexpr double FX50 = 1125899906842624.0;        // 2^50: fixed-point scale of the final stage
constexpr uint32_t KEY_MIN_FINITE = 0x00800000u;   // key(-FLT_MAX); key(-inf) is one below
constexpr uint32_t KEY_POS_INF = 0xFF800000u;      // key(+inf)
constexpr float FX_SCALE = 1099511627776.0f;       // 2^40: fixed-point scale of masses
constexpr double LN2_40 = 27.725887222397812;      // 40 ln 2

struct SampleArgs {
    const void *logits;
    int32_t B, V;
    int64_t row_stride;
    const float *temperature;
    const int32_t *top_k;
    const float *top_p, *min_p, *rep, *pres, *freq;
    const int32_t *hist_ids, *hist_off;
    const uint64_t *seeds;
    uint64_t step;
    uint32_t row_base;
    uint32_t flags;
    int32_t *out_tokens;
    float *out_logprobs;
    int32_t num_top;
    int32_t *out_top_ids;
    float *out_top_logprobs;
    int32_t *out_num_kept, *out_num_topk;
    int32_t dbg_cap;
    int32_t *dbg_topk_ids;
    uint32_t *out_row_status;
    uint32_t *ws_counts;        // global scratch for history counts of rows with many distinct ids
    int64_t ws_counts_cap;      // entries
};

// ------------------------------------------------------------------ scalar helpers

__device__ __forceinline__ uint32_t key_of(float z) {
    uint32_t b = __float_as_uint(z);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float unkey(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}
__device__ __forceinline__ u64 comp_of(uint32_t key, int i) {
    return ((u64)key << 32) | (uint32_t)(~(uint32_t)i);
}
__device__ __forceinline__ int comp_idx(u64 c) { return (int)(~(uint32_t)c); }

// Philox4x32-10 with the sampler's keying: counter (t>>2, R, step lo, step hi), key (seed lo, seed hi).
__device__ __forceinline__ uint32_t race_word(uint64_t seed, uint32_t R, uint64_t step, int t) {
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    uint32_t c0 = (uint32_t)t >> 2, c1 = R, c2 = (uint32_t)step, c3 = (uint32_t)(step >> 32);
    uint32_t k0 = (uint32_t)seed, k1 = (uint32_t)(seed >> 32);
#pragma unroll
    for (int i = 0; i < 10; ++i) {
        uint32_t h0 = __umulhi(M0, c0), l0 = M0 * c0;
        uint32_t h1 = __umulhi(M1, c2), l1 = M1 * c2;
        c0 = h1 ^ c1 ^ k0; c1 = l1; c2 = h0 ^ c3 ^ k1; c3 = l0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    int wsel = t & 3;
    return wsel == 0 ? c0 : wsel == 1 ? c1 : wsel == 2 ? c2 : c3;
}

// -ln(E) for E = -log1p(-v), v = (w + 1/2) 2^-32, in fp32.  The half of the range near
// v = 1 is evaluated from 1 - v = (~w + 1/2) 2^-32 so both ends keep full relative accuracy.
__device__ __forceinline__ float neg_log_exp1_f32(uint32_t w) {
    float E;
    if (w < 0x80000000u) {
        float v = __fmaf_rn((float)w, 2.3283064365386963e-10f, 1.1641532182693481e-10f);
        E = -log1pf(-v);
    } else {
        float omv = __fmaf_rn((float)(~w), 2.3283064365386963e-10f, 1.1641532182693481e-10f);
        E = -logf(omv);
    }
    return -logf(E);
}
__device__ __forceinline__ double neg_log_exp1_f64(uint32_t w) {
    double v = ((double)w + 0.5) * (1.0 / 4294967296.0);
    return -log(-log1p(-v));
}

__device__ __forceinline__ uint32_t orderable_f32(float g) { return key_of(g); }

// fixed-point mass of an element at distance d = z - zmax <= 0 (deterministic integer sums)
__device__ __forceinline__ u64 mass_fx(float d) {
    return __float2ull_rn(expf(d) * FX_SCALE);
}

// ------------------------------------------------------------------ block primitives

struct BlockScratch {
    u64 red[NWARPS];
    u64 red2[NWARPS];
    u64 bcast[4];
    uint32_t found_digit, found_cnt;
    u64 found_above;
    uint32_t list_cnt;
    uint32_t cand_cnt, overflow, runmax;
};

__device__ __forceinline__ u64 warp_max_u64(u64 v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { u64 t = __shfl_xor_sync(0xFFFFFFFFu, v, o); v = t > v ? t : v; }
    return v;
}
__device__ __forceinline__ u64 warp_sum_u64(u64 v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}
// all threads get the result; contains two barriers
__device__ u64 block_max_u64(BlockScratch &s, u64 v) {
    v = warp_max_u64(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s.red[threadIdx.x >> 5] = v;
    __syncthreads();
    u64 r = s.red[0];
#pragma unroll
    for (int w = 1; w < NWARPS; ++w) { u64 t = s.red[w]; r = t > r ? t : r; }
    return r;
}
__device__ u64 block_sum_u64(BlockScratch &s, u64 v) {
    v = warp_sum_u64(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s.red[threadIdx.x >> 5] = v;
    __syncthreads();
    u64 r = 0;
#pragma unroll
    for (int w = 0; w < NWARPS; ++w) r += s.red[w];
    return r;
}
// exclusive prefix sum over threads in thread order; also returns the block total
__device__ u64 block_exscan_u64(BlockScratch &s, u64 v, u64 &total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    u64 inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { u64 t = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += t; }
    __syncthreads();
    if (lane == 31) s.red2[wid] = inc;
    __syncthreads();
    u64 base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < NWARPS; ++w) { u64 t = s.red2[w]; if (w < wid) base += t; tot += t; }
    total = tot;
    return base + inc - v;
}

// ------------------------------------------------------------------ row context

struct RowCtx {
    const void *row;       // first logit of the row
    int V;
    float invT, r, p, f;
    bool has_hist;
    const uint32_t *bitmap;   // V bits (+1 pad word): token appears in the history
    const uint32_t *coarse;   // exclusive popcount prefix per 8 bitmap words
    const uint32_t *counts;   // occurrence count per distinct id, indexed by rank in the bitmap
};

__device__ __forceinline__ uint32_t hist_rank(const RowCtx &c, int i) {
    int w = i >> 5, cb = w >> 3;
    uint32_t r = c.coarse[cb];
    for (int ww = cb << 3; ww < w; ++ww) r += __popc(c.bitmap[ww]);
    r += __popc(c.bitmap[w] & ((1u << (i & 31)) - 1u));
    return r;
}

// penalties: each line is one rounded fp32 operation
__device__ __forceinline__ float penalise(const RowCtx &c, int i, float x) {
    uint32_t cnt = c.counts[hist_rank(c, i)];
    float a = (x > 0.0f) ? __fdiv_rn(x, c.r) : __fmul_rn(x, c.r);
    float t = __fmul_rn(c.f, __uint2float_rn(cnt));
    a = __fsub_rn(a, t);
    a = __fsub_rn(a, c.p);
    return a;
}

template <int DT> struct Elem;
template <> struct Elem<ALBIREO_F32> {
    static constexpr int SIZE = 4, PER_VEC = 4;
    static __device__ __forceinline__ float load(const void *row, int i) { return __ldg((const float *)row + i); }
    static __device__ __forceinline__ float get(const uint4 &q, int e) {
        return __uint_as_float(e == 0 ? q.x : e == 1 ? q.y : e == 2 ? q.z : q.w);
    }
};
template <> struct Elem<ALBIREO_BF16> {
    static constexpr int SIZE = 2, PER_VEC = 8;
    static __device__ __forceinline__ float load(const void *row, int i) {
        return __uint_as_float(((uint32_t)__ldg((const unsigned short *)row + i)) << 16);
    }
    static __device__ __forceinline__ float get(const uint4 &q, int e) {
        uint32_t w = (e >> 1) == 0 ? q.x : (e >> 1) == 1 ? q.y : (e >> 1) == 2 ? q.z : q.w;
        return __uint_as_float((e & 1) ? (w & 0xFFFF0000u) : (w << 16));
    }
};

__device__ __forceinline__ float score_of(const RowCtx &c, int i, float x) {
    float a = x;
    if (c.has_hist && ((c.bitmap[i >> 5] >> (i & 31)) & 1u)) a = penalise(c, i, x);
    return __fmul_rn(a, c.invT);
}

// Calls fn(i, z_i) for every element of the row (each thread a strided share).
// 16-byte vector loads over the aligned middle of the row, scalar head and tail.
template <int DT, class F>
__device__ __forceinline__ void for_each_score(const RowCtx &c, F &&fn) {
    typedef Elem<DT> E;
    const int V = c.V;
    const uintptr_t addr = (uintptr_t)c.row;
    int head = (int)(((16u - (uint32_t)(addr & 15u)) & 15u) / E::SIZE);
    if (head > V) head = V;
    const int nvec = (V - head) / E::PER_VEC;
    const uint4 *vp = (const uint4 *)((const char *)c.row + (size_t)head * E::SIZE);
    for (int v = threadIdx.x; v < nvec; v += NT) {
        const uint4 q = __ldg(vp + v);
        const int i0 = head + v * E::PER_VEC;
        uint32_t m = 0;
        if (c.has_hist) {
            m = __funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31) & ((1u << E::PER_VEC) - 1u);
        }
#pragma unroll
        for (int e = 0; e < E::PER_VEC; ++e) {
            float x = E::get(q, e);
            float a = x;
            if (m & (1u << e)) a = penalise(c, i0 + e, x);
            fn(i0 + e, __fmul_rn(a, c.invT));
        }
    }
    for (int i = threadIdx.x; i < head; i += NT) fn(i, score_of(c, i, E::load(c.row, i)));
    for (int i = head + nvec * E::PER_VEC + threadIdx.x; i < V; i += NT) fn(i, score_of(c, i, E::load(c.row, i)));
}

// ------------------------------------------------------------------ history -> bitmap + counts

struct HistSmem {
    uint32_t *bitmap;   // nwords + 1
    uint32_t *coarse;   // ncoarse + 1
    uint32_t *counts;   // CNT_CAP
};

// Builds the per-row penalty tables.  Returns false (penalties skipped) if the distinct
// ids fit neither on chip nor in the caller's workspace.
__device__ bool build_history(BlockScratch &s, const HistSmem &hs, RowCtx &c, const int32_t *ids, int len,
                              uint32_t *ws, int64_t ws_cap, int64_t ws_off) {
    const int V = c.V;
    const int nwords = (V + 31) >> 5, ncoarse = (nwords + 7) >> 3;
    for (int w = threadIdx.x; w <= nwords; w += NT) hs.bitmap[w] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < len; j += NT) {
        int t = __ldg(ids + j);
        if (t >= 0 && t < V) atomicOr(&hs.bitmap[t >> 5], 1u << (t & 31));
    }
    __syncthreads();
    // coarse exclusive prefix: one entry per 8 words; ncoarse <= 2048 for V <= 2^19
    u64 carry = 0;
    for (int base = 0; base < ncoarse; base += NT) {
        int cb = base + threadIdx.x;
        uint32_t pc = 0;
        if (cb < ncoarse) {
            for (int w = cb << 3; w < min(nwords, (cb << 3) + 8); ++w) pc += __popc(hs.bitmap[w]);
        }
        u64 tot;
        u64 ex = block_exscan_u64(s, pc, tot);
        if (cb < ncoarse) hs.coarse[cb] = (uint32_t)(carry + ex);
        carry += tot;
    }
    const uint32_t U = (uint32_t)carry;     // distinct valid ids
    uint32_t *cnt;
    bool ok = true;
    if (U <= CNT_CAP) cnt = hs.counts;
    else if (ws && ws_off + (int64_t)U <= ws_cap) cnt = ws + ws_off;
    else { cnt = nullptr; ok = false; }
    c.bitmap = hs.bitmap; c.coarse = hs.coarse; c.counts = cnt;
    if (!ok) return false;
    for (uint32_t u = threadIdx.x; u < U; u += NT) cnt[u] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < len; j += NT) {
        int t = __ldg(ids + j);
        if (t >= 0 && t < V) atomicAdd(&cnt[hist_rank(c, t)], 1u);
    }
    __syncthreads();
    return true;
}

// ------------------------------------------------------------------ general path: radix selection

struct HistBins {
    uint32_t *cnt;   // HIST_BINS
    u64 *mass;       // HIST_BINS
};

__constant__ int LVL_SHIFT[6] = {53, 42, 32, 21, 10, 0};
__constant__ int LVL_BITS[6] = {11, 11, 10, 11, 11, 10};

// Scans bins from the highest digit down and finds the bin where the running total first
// reaches `target` (target >= 1, <= grand total).  use_mass selects which histogram steers.
// Returns digit, the total strictly above the bin, and the bin's element count.
__device__ void find_bin(BlockScratch &s, const HistBins &h, int nbins, bool use_mass, u64 target,
                         uint32_t &digit, u64 &above, uint32_t &bin_cnt) {
    // thread t owns bins [nbins - per*(t+1), nbins - per*t), visited from the top
    const int per = (nbins + NT - 1) / NT;
    u64 local = 0;
    for (int q = 0; q < per; ++q) {
        int bin = nbins - 1 - (threadIdx.x * per + q);
        if (bin >= 0) local += use_mass ? h.mass[bin] : (u64)h.cnt[bin];
    }
    u64 tot;
    u64 run = block_exscan_u64(s, local, tot);
    if (threadIdx.x == 0) { s.found_digit = 0xFFFFFFFFu; s.found_cnt = 0; s.found_above = 0; }
    __syncthreads();
    if (run < target && target <= run + local) {
        for (int q = 0; q < per; ++q) {
            int bin = nbins - 1 - (threadIdx.x * per + q);
            if (bin < 0) break;
            u64 v = use_mass ? h.mass[bin] : (u64)h.cnt[bin];
            if (run < target && target <= run + v) {
                s.found_digit = (uint32_t)bin; s.found_above = run; s.found_cnt = h.cnt[bin];
                break;
            }
            run += v;
        }
    }
    __syncthreads();
    digit = s.found_digit; above = s.found_above; bin_cnt = s.found_cnt;
}

// Selection by count: returns the composite of the `rank`-th largest element (1-based)
// among { C >= lo } whose top bits (above level `lvl0`) equal `prefix`.
// Precondition: 1 <= rank <= number of such elements.
template <int DT>
__device__ u64 select_by_count(BlockScratch &s, const HistBins &h, const RowCtx &c, u64 lo, u64 rank,
                               int lvl0, u64 prefix) {
    for (int lvl = lvl0; lvl < 6; ++lvl) {
        const int shift = LVL_SHIFT[lvl], bits = LVL_BITS[lvl], nbins = 1 << bits;
        if (lvl == 3 && c.V <= (1 << 21)) { prefix = (prefix << 11) | 0x7FFu; continue; }  // ~id has these bits all set
        for (int bnum = threadIdx.x; bnum < nbins; bnum += NT) h.cnt[bnum] = 0;
        __syncthreads();
        const int up = shift + bits;
        for_each_score<DT>(c, [&](int i, float z) {
            u64 C = comp_of(key_of(z), i);
            bool in = C >= lo && (up >= 64 || (C >> up) == prefix);
            if (in) atomicAdd(&h.cnt[(uint32_t)(C >> shift) & (nbins - 1)], 1u);
        });
        __syncthreads();
        uint32_t digit, bin_cnt; u64 above;
        find_bin(s, h, nbins, false, rank, digit, above, bin_cnt);
        if (digit == 0xFFFFFFFFu) return lo;            // precondition violated; keep everything
        rank -= above;
        prefix = (prefix << bits) | digit;
        if (rank == bin_cnt) {                           // the whole bin is taken
            u64 t = prefix << shift;
            return t > lo ? t : lo;
        }
    }
    return prefix;
}

// Selection by mass: smallest prefix of { C >= lo } whose mass reaches top_p times the
// mass of the whole set.  Returns its composite threshold.
template <int DT>
__device__ u64 select_by_mass(BlockScratch &s, const HistBins &h, const RowCtx &c, u64 lo, float zmax, float top_p) {
    u64 prefix = 0, target = 0;
    uint32_t bin_cnt = 0;
    for (int lvl = 0; lvl < 3; ++lvl) {
        const int shift = LVL_SHIFT[lvl], bits = LVL_BITS[lvl], nbins = 1 << bits;
        for (int bnum = threadIdx.x; bnum < nbins; bnum += NT) { h.cnt[bnum] = 0; h.mass[bnum] = 0; }
        __syncthreads();
        const int up = shift + bits;
        for_each_score<DT>(c, [&](int i, float z) {
            u64 C = comp_of(key_of(z), i);
            bool in = C >= lo && (up >= 64 || (C >> up) == prefix);
            if (in) {
                uint32_t d = (uint32_t)(C >> shift) & (nbins - 1);
                atomicAdd(&h.cnt[d], 1u);
                atomicAdd(&h.mass[d], mass_fx(__fsub_rn(z, zmax)));
            }
        });
        __syncthreads();
        if (lvl == 0) {
            u64 local = 0;
            for (int bnum = threadIdx.x; bnum < nbins; bnum += NT) local += h.mass[bnum];
            u64 total = block_sum_u64(s, local);
            double t = ceil((double)top_p * (double)total);
            target = t <= 1.0 ? 1ull : (u64)t;
            if (target > total) target = total;
            if (target < 1) target = 1;
        }
        uint32_t digit; u64 above;
        find_bin(s, h, nbins, true, target, digit, above, bin_cnt);
        if (digit == 0xFFFFFFFFu) return lo;
        target -= above;
        prefix = (prefix << bits) | digit;
    }
    // prefix is now a full key; bin_cnt ties share one mass value each
    const uint32_t tkey = (uint32_t)prefix;
    u64 e1 = mass_fx(__fsub_rn(unkey(tkey), zmax));
    u64 m = e1 ? (target + e1 - 1) / e1 : bin_cnt;
    if (m < 1) m = 1;
    u64 tie_lo = ((u64)tkey << 32) > lo ? ((u64)tkey << 32) : lo;
    if (m >= bin_cnt) return tie_lo;
    return select_by_count<DT>(s, h, c, tie_lo, m, 3, (u64)tkey);
}

struct RowParams {
    float T, top_p, min_p;
    int32_t top_k;
    uint64_t seed;
    uint32_t R;
    bool greedy;
};

struct RowOut {
    int32_t token; float logprob; int32_t n_keep, n_topk; uint32_t status;
};

// smallest fp32 z with (double)z - (double)zmax >= ln(min_p), as an order key
__device__ uint32_t minp_key(float zmax, float min_p) {
    const double thr = log((double)min_p);
    const double zm = (double)zmax;
    float z = (float)(zm + thr);
    // settle on the exact boundary (a handful of ulp steps at most)
    for (int it = 0; it < 64 && !((double)z - zm >= thr); ++it) z = unkey(key_of(z) + 1);
    for (int it = 0; it < 64; ++it) {
        uint32_t k = key_of(z);
        if (k <= KEY_MIN_FINITE) break;
        float zd = unkey(k - 1);
        if ((double)zd - zm >= thr) z = zd; else break;
    }
    uint32_t k = key_of(z);
    return k < KEY_MIN_FINITE ? KEY_MIN_FINITE : k;
}

// Gathers { C >= thr } (at most cap of them) into list[], sorted best first.  list must
// hold cap entries.  Returns the number gathered (elements beyond cap are dropped).
template <int DT>
__device__ int gather_sorted(BlockScratch &s, const RowCtx &c, u64 thr, u64 *list, u64 *tmp, int cap) {
    if (threadIdx.x == 0) s.list_cnt = 0;
    __syncthreads();
    for_each_score<DT>(c, [&](int i, float z) {
        u64 C = comp_of(key_of(z), i);
        if (C >= thr) { uint32_t slot = atomicAdd(&s.list_cnt, 1u); if (slot < (uint32_t)cap) tmp[slot] = C; }
    });
    __syncthreads();
    int n = min((int)s.list_cnt, cap);
    for (int a = threadIdx.x; a < n; a += NT) {
        u64 C = tmp[a]; int rank = 0;
        for (int b2 = 0; b2 < n; ++b2) rank += tmp[b2] > C;
        list[rank] = C;
    }
    __syncthreads();
    return n;
}

template <int DT>
__device__ void general_path(BlockScratch &s, const HistBins &h, const RowCtx &c, const RowParams &rp,
                             const SampleArgs &a, int b, RowOut &out) {
    const int V = c.V;
    // pass 0: the top element and the number of finite scores
    u64 best = 0; uint32_t nfin_local = 0;
    for_each_score<DT>(c, [&](int i, float z) {
        uint32_t k = key_of(z);
        u64 C = comp_of(k, i);
        best = C > best ? C : best;
        nfin_local += (k >= KEY_MIN_FINITE && k < KEY_POS_INF);
    });
    const u64 Ctop = block_max_u64(s, best);
    const u64 n_fin = block_sum_u64(s, nfin_local);
    const float zmax = unkey((uint32_t)(Ctop >> 32));
    out.status |= ALBIREO_ROW_GENERAL_PATH;

    if (rp.greedy || n_fin <= 1) {
        out.token = comp_idx(Ctop); out.logprob = 0.0f; out.n_keep = 1; out.n_topk = 1;
        if (a.dbg_topk_ids && a.dbg_cap >= 1 && threadIdx.x == 0) a.dbg_topk_ids[(int64_t)b * a.dbg_cap] = out.token;
        if (a.num_top > 0 && threadIdx.x == 0) {
            a.out_top_ids[(int64_t)b * a.num_top] = out.token;
            a.out_top_logprobs[(int64_t)b * a.num_top] = 0.0f;
        }
        return;
    }

    // top-k stage
    const u64 Cfin = (u64)KEY_MIN_FINITE << 32;
    u64 C1 = Cfin;
    u64 n_topk = n_fin;
    if (rp.top_k >= 1 && rp.top_k < V && (u64)rp.top_k < n_fin) {
        n_topk = (u64)rp.top_k;
        C1 = select_by_count<DT>(s, h, c, Cfin, n_topk, 0, 0);
    }
    out.n_topk = (int32_t)n_topk;
    if (a.dbg_topk_ids && rp.top_k >= 1 && rp.top_k < V && n_topk <= (u64)a.dbg_cap) {
        if (threadIdx.x == 0) s.list_cnt = 0;
        __syncthreads();
        int32_t *dst = a.dbg_topk_ids + (int64_t)b * a.dbg_cap;
        for_each_score<DT>(c, [&](int i, float z) {
            if (comp_of(key_of(z), i) >= C1) { uint32_t slot = atomicAdd(&s.list_cnt, 1u); if (slot < (uint32_t)a.dbg_cap) dst[slot] = i; }
        });
        __syncthreads();
    }
    // min-p: a value threshold, never above the top element
    if (rp.min_p > 0.0f) {
        u64 Cm = (u64)minp_key(zmax, rp.min_p) << 32;
        if (Cm > Ctop) Cm = Ctop;
        if (Cm > C1) C1 = Cm;
    }
    // top-p on the mass of the survivors
    u64 C2 = C1;
    if (rp.top_p < 1.0f) C2 = select_by_mass<DT>(s, h, c, C1, zmax, rp.top_p);

    // final pass: mass of the kept set, its size, and the race
    u64 S_local = 0, n_local = 0, g_best = 0;
    for_each_score<DT>(c, [&](int i, float z) {
        u64 C = comp_of(key_of(z), i);
        if (C >= C2) {
            float d = __fsub_rn(z, zmax);
            S_local += mass_fx(d);
            n_local += 1;
            float g = d + neg_log_exp1_f32(race_word(rp.seed, rp.R, a.step, i));
            u64 G = ((u64)orderable_f32(g) << 32) | (uint32_t)(~(uint32_t)i);
            g_best = G > g_best ? G : g_best;
        }
    });
    const u64 S_fx = block_sum_u64(s, S_local);
    const u64 n_keep = block_sum_u64(s, n_local);
    const u64 G = block_max_u64(s, g_best);
    const int tok = comp_idx(G);
    const double lnS = log((double)S_fx) - LN2_40;
    float z_tok = score_of(c, tok, Elem<DT>::load(c.row, tok));
    out.token = (n_keep == 1) ? comp_idx(Ctop) : tok;
    out.logprob = (n_keep == 1) ? 0.0f : (float)(((double)z_tok - (double)zmax) - lnS);
    out.n_keep = (int32_t)n_keep;

    if (a.num_top > 0) {
        // first min(num_top, n_keep) entries of the kept set, in order
        u64 *list = (u64 *)h.mass;                 // histograms are free again: reuse as two lists
        u64 *tmp = list + ALBIREO_MAX_NUM_TOP;
        u64 want = n_keep < (u64)a.num_top ? n_keep : (u64)a.num_top;
        u64 CN = (want == n_keep) ? C2 : select_by_count<DT>(s, h, c, C2, want, 0, 0);
        __syncthreads();
        int n = gather_sorted<DT>(s, c, CN, list, tmp, ALBIREO_MAX_NUM_TOP);
        for (int j = threadIdx.x; j < a.num_top; j += NT) {
            int64_t q = (int64_t)b * a.num_top + j;
            if (j < n) {
                int id = comp_idx(list[j]);
                float zj = unkey((uint32_t)(list[j] >> 32));
                a.out_top_ids[q] = id;
                a.out_top_logprobs[q] = (float)(((double)zj - (double)zmax) - lnS);
            } else {
                a.out_top_ids[q] = -1;
                a.out_top_logprobs[q] = __uint_as_float(0xFF800000u);
            }
        }
        __syncthreads();
    }
}


// ------------------------------------------------------------------ candidate path
//
// One streaming pass over the row.  A conservative threshold tau (an order key) is kept
// such that every element of the final kept set has key >= tau: the k-th largest key
// among the candidates seen so far (top-k), and/or the min-p floor below the running
// maximum.  Elements below tau are dropped by a cheap vector test; the rest are checked
// exactly and appended to a small on-chip candidate list, which is then sorted and cut.
// Penalised tokens never enter through the stream (their raw value is not their score):
// they are evaluated from the history bitmap after the stream.

struct CandSmem {
    u64 *cand;        // CAND_CAP composites
    u64 *sorted;      // SORT_MAX composites, best first
    uint32_t *hist;   // 256 bins
};

__device__ __forceinline__ void cand_append(BlockScratch &s, u64 *cand, u64 C) {
    uint32_t slot = atomicAdd(&s.cand_cnt, 1u);
    if (slot < (uint32_t)CAND_CAP) cand[slot] = C; else s.overflow = 1u;
    atomicMax(&s.runmax, (uint32_t)(C >> 32));
}

// k-th largest key (1-based) among cand[0..n), n >= k: 8-bit radix select.  Uniform result.
__device__ uint32_t cand_select_key(BlockScratch &s, const CandSmem &cs, int n, int k) {
    uint32_t prefix = 0;
    uint32_t rank = (uint32_t)k;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (threadIdx.x < 256) cs.hist[threadIdx.x] = 0;
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += NT) {
            uint32_t key = (uint32_t)(cs.cand[i] >> 32);
            if (pass == 0 || (key >> (shift + 8)) == prefix) atomicAdd(&cs.hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (threadIdx.x < 32) {
            const int lane = threadIdx.x;
            uint32_t local = 0;
#pragma unroll
            for (int q = 0; q < 8; ++q) local += cs.hist[255 - (lane * 8 + q)];
            uint32_t inc = local;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += t; }
            uint32_t run = inc - local;
            if (run < rank && rank <= run + local) {
                for (int q = 0; q < 8; ++q) {
                    uint32_t v = cs.hist[255 - (lane * 8 + q)];
                    if (rank <= run + v) { s.found_digit = 255 - (lane * 8 + q); s.found_above = run; break; }
                    run += v;
                }
            }
        }
        __syncthreads();
        rank -= (uint32_t)s.found_above;
        prefix = (prefix << 8) | s.found_digit;
    }
    return prefix;
}

// keeps the candidates with key >= tkey; returns the new count (uniform)
__device__ int cand_compact(BlockScratch &s, const CandSmem &cs, int n, uint32_t tkey) {
    constexpr int PER = CAND_CAP / NT;
    u64 mine[PER];
#pragma unroll
    for (int q = 0; q < PER; ++q) {
        int i = threadIdx.x + q * NT;
        mine[q] = (i < n) ? cs.cand[i] : 0ull;
    }
    __syncthreads();
    if (threadIdx.x == 0) s.cand_cnt = 0;
    __syncthreads();
#pragma unroll
    for (int q = 0; q < PER; ++q) {
        if ((uint32_t)(mine[q] >> 32) >= tkey && mine[q] != 0ull) {
            uint32_t slot = atomicAdd(&s.cand_cnt, 1u);
            cs.cand[slot] = mine[q];
        }
    }
    __syncthreads();
    return (int)s.cand_cnt;
}

// Vector pre-test per dtype.  RawThr is the threshold in the domain the test runs in:
// bf16: the smallest raw bf16 whose score has key >= tau (packed twice); fp32: unkey(tau).
template <int DT> struct VecTest;
template <> struct VecTest<ALBIREO_BF16> {
    static __device__ uint32_t raw_threshold(uint32_t tau_key, float invT) {
        const float tz = unkey(tau_key);
        const float xg = __fdiv_rn(tz, invT);
        const uint32_t b16 = __float_as_uint(xg) >> 16;
        uint32_t k16 = (b16 & 0x8000u) ? (~b16 & 0xFFFFu) : (b16 | 0x8000u);
        auto bits_of = [](uint32_t kk) { return (kk & 0x8000u) ? (kk & 0x7FFFu) : (~kk & 0xFFFFu); };
        auto passes = [&](uint32_t kk) {
            float x = __uint_as_float(bits_of(kk) << 16);
            return key_of(__fmul_rn(x, invT)) >= tau_key;
        };
        if (k16 < 0x0080u) k16 = 0x0080u;
        if (k16 > 0xFF7Fu) k16 = 0xFF7Fu;
        int it = 0;
        while (it < 16 && k16 > 0x0080u && passes(k16)) { --k16; ++it; }
        while (it < 32 && k16 < 0xFF7Fu && !passes(k16)) { ++k16; ++it; }
        const bool ok = passes(k16) && (k16 == 0x0080u || !passes(k16 - 1));
        const uint32_t b = ok ? bits_of(k16) : 0xFF80u;     // not settled: let everything through
        return b | (b << 16);
    }
    static __device__ __forceinline__ bool may_pass(const uint4 &q, uint32_t thr, float) {
        __nv_bfloat162 a = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&q.x), *reinterpret_cast<const __nv_bfloat162 *>(&q.y));
        __nv_bfloat162 b2 = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&q.z), *reinterpret_cast<const __nv_bfloat162 *>(&q.w));
        a = __hmax2(a, b2);
        return __hge2_mask(a, *reinterpret_cast<const __nv_bfloat162 *>(&thr)) != 0u;
    }
    static __device__ __forceinline__ uint4 fill() { return make_uint4(0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u, 0xFF80FF80u); }
};
template <> struct VecTest<ALBIREO_F32> {
    static __device__ uint32_t raw_threshold(uint32_t tau_key, float) { return __float_as_uint(unkey(tau_key)); }
    static __device__ __forceinline__ bool may_pass(const uint4 &q, uint32_t thr, float invT) {
        float m = fmaxf(fmaxf(__fmul_rn(__uint_as_float(q.x), invT), __fmul_rn(__uint_as_float(q.y), invT)),
                        fmaxf(__fmul_rn(__uint_as_float(q.z), invT), __fmul_rn(__uint_as_float(q.w), invT)));
        return m >= __uint_as_float(thr);
    }
    static __device__ __forceinline__ uint4 fill() { return make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u); }
};

// exact check of one vector's unpenalised elements against tau; appends survivors
template <int DT>
__device__ __noinline__ void slow_vector(BlockScratch &s, u64 *cand, const RowCtx &c, uint4 q, int i0,
                                         uint32_t tau_key, u64 skip) {
    typedef Elem<DT> E;
    uint32_t m = 0;
    if (c.has_hist) m = __funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31);
#pragma unroll
    for (int e = 0; e < E::PER_VEC; ++e) {
        if (m & (1u << e)) continue;
        uint32_t key = key_of(__fmul_rn(E::get(q, e), c.invT));
        u64 C = comp_of(key, i0 + e);
        if (key >= tau_key && C != skip) cand_append(s, cand, C);
    }
}

// Returns false if the row must be handled by the general path instead.
template <int DT>
__device__ bool candidate_path(BlockScratch &s, const CandSmem &cs, const RowCtx &c, const RowParams &rp,
                               const SampleArgs &a, int b, RowOut &out) {
    typedef Elem<DT> E;
    typedef VecTest<DT> T;
    const int V = c.V;
    const int k = rp.greedy ? 1 : rp.top_k;
    const bool has_topk = rp.greedy || (k >= 1 && k < V);
    const bool has_minp = !rp.greedy && rp.min_p > 0.0f;
    if (has_topk && k > KA_MAX) return false;
    if (!has_topk && !has_minp) return false;
    // with the debug id list requested, keep the stream's threshold purely top-k so that the
    // top-k stage's set is known exactly
    const bool stream_minp = has_minp && !(has_topk && a.dbg_topk_ids != nullptr);
    const double ln_minp = has_minp ? log((double)rp.min_p) : 0.0;

    if (threadIdx.x == 0) { s.cand_cnt = 0; s.overflow = 0; s.runmax = 0; }
    __syncthreads();

    const uintptr_t addr = (uintptr_t)c.row;
    int head = (int)(((16u - (uint32_t)(addr & 15u)) & 15u) / E::SIZE);
    if (head > V) head = V;
    const int nvec = (V - head) / E::PER_VEC;
    const uint4 *vp = (const uint4 *)((const char *)c.row + (size_t)head * E::SIZE);
    const int ntiles = (nvec + NT * TILE_VECS - 1) / (NT * TILE_VECS);

    uint32_t tau_key = KEY_MIN_FINITE;
    uint32_t thr = T::raw_threshold(tau_key, c.invT);
    uint32_t seen_max = 0;

    auto floor_from_max = [&](uint32_t maxkey) -> uint32_t {
        // a key no larger than the key of the smallest score that passes min-p under this maximum
        return minp_key(unkey(maxkey), rp.min_p);
    };

    uint4 cur[TILE_VECS], nxt[TILE_VECS];
#pragma unroll
    for (int u = 0; u < TILE_VECS; ++u) {
        int v = u * NT + threadIdx.x;
        cur[u] = (v < nvec) ? __ldg(vp + v) : T::fill();
    }
    for (int tile = 0; tile < ntiles; ++tile) {
        const int vbase = tile * NT * TILE_VECS;
        if (tile + 1 < ntiles) {
#pragma unroll
            for (int u = 0; u < TILE_VECS; ++u) {
                int v = vbase + NT * TILE_VECS + u * NT + threadIdx.x;
                nxt[u] = (v < nvec) ? __ldg(vp + v) : T::fill();
            }
        }
        u64 own = 0;
        if (tile == 0) {
            // warm-up: every thread contributes its best unpenalised element; the k-th largest
            // of these is a valid lower bound of the row's k-th largest score
#pragma unroll
            for (int u = 0; u < TILE_VECS; ++u) {
                const int i0 = head + (vbase + u * NT + threadIdx.x) * E::PER_VEC;
                uint32_t m = 0;
                if (c.has_hist && i0 < V) m = __funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31);
#pragma unroll
                for (int e = 0; e < E::PER_VEC; ++e) {
                    uint32_t key = key_of(__fmul_rn(E::get(cur[u], e), c.invT));
                    u64 C = comp_of(key, i0 + e);
                    if (!(m & (1u << e)) && key >= KEY_MIN_FINITE && C > own) own = C;
                }
            }
            if (own) cand_append(s, cs.cand, own);
            __syncthreads();
            int n = (int)s.cand_cnt;
            uint32_t rmax = s.runmax;
            __syncthreads();
            if (has_topk && n >= k) tau_key = cand_select_key(s, cs, n, k);
            if (stream_minp && rmax) { uint32_t f = floor_from_max(rmax); tau_key = f > tau_key ? f : tau_key; }
            seen_max = rmax;
            thr = T::raw_threshold(tau_key, c.invT);
        }
#pragma unroll
        for (int u = 0; u < TILE_VECS; ++u) {
            const int v = vbase + u * NT + threadIdx.x;
            if (v < nvec && T::may_pass(cur[u], thr, c.invT))
                slow_vector<DT>(s, cs.cand, c, cur[u], head + v * E::PER_VEC, tau_key, own);
        }
        __syncthreads();                       // every append of this tile is done
        int n = (int)s.cand_cnt;
        const uint32_t ovf = s.overflow, rmax = s.runmax;
        __syncthreads();                       // nobody appends again before all have read
        if (ovf) return false;
        bool changed = false;
        if (has_topk && n >= k && (n >= 2 * k + 32 || n > CAND_CAP / 2 || tile == 0)) {
            uint32_t t = cand_select_key(s, cs, n, k);
            if (t > tau_key) { tau_key = t; changed = true; }
            n = cand_compact(s, cs, n, tau_key);
        }
        if (stream_minp && rmax != seen_max) {
            seen_max = rmax;
            uint32_t f = floor_from_max(rmax);
            if (f > tau_key) { tau_key = f; changed = true; }
        }
        if (!has_topk && n > CAND_CAP / 2) n = cand_compact(s, cs, n, tau_key);
        if (changed) thr = T::raw_threshold(tau_key, c.invT);
#pragma unroll
        for (int u = 0; u < TILE_VECS; ++u) cur[u] = nxt[u];
    }
    // scalar head and tail of a row that is not 16-byte aligned / not a whole number of vectors
    {
        const int tail0 = head + nvec * E::PER_VEC;
        const int nscal = head + (V - tail0);
        for (int q = threadIdx.x; q < nscal; q += NT) {
            int i = q < head ? q : tail0 + (q - head);
            if (c.has_hist && ((c.bitmap[i >> 5] >> (i & 31)) & 1u)) continue;
            uint32_t key = key_of(__fmul_rn(E::load(c.row, i), c.invT));
            if (key >= tau_key) cand_append(s, cs.cand, comp_of(key, i));
        }
    }
    // penalised tokens, straight from the history bitmap
    if (c.has_hist) {
        const int nwords = (V + 31) >> 5;
        for (int w = threadIdx.x; w < nwords; w += NT) {
            uint32_t bits = c.bitmap[w];
            if (!bits) continue;
            uint32_t r = c.coarse[w >> 3];
            for (int ww = (w >> 3) << 3; ww < w; ++ww) r += __popc(c.bitmap[ww]);
            while (bits) {
                int bit = __ffs(bits) - 1;
                bits &= bits - 1;
                int i = (w << 5) + bit;
                float x = E::load(c.row, i);
                uint32_t cnt = c.counts[r++];
                float av = (x > 0.0f) ? __fdiv_rn(x, c.r) : __fmul_rn(x, c.r);
                av = __fsub_rn(av, __fmul_rn(c.f, __uint2float_rn(cnt)));
                av = __fsub_rn(av, c.p);
                uint32_t key = key_of(__fmul_rn(av, c.invT));
                if (key >= tau_key) cand_append(s, cs.cand, comp_of(key, i));
            }
        }
    }
    __syncthreads();
    int n = (int)s.cand_cnt;
    const uint32_t ovf = s.overflow;
    const uint32_t kmax = s.runmax;
    __syncthreads();
    if (ovf || n < 1) return false;

    // exact top-k threshold, then the exact min-p floor for rows without a top-k
    bool topk_exact_known = true;      // is min(k, #finite) known without counting?
    if (has_topk) {
        if (n > k) {
            uint32_t t = cand_select_key(s, cs, n, k);
            n = cand_compact(s, cs, n, t);
        } else if (n < k && stream_minp) {
            topk_exact_known = false;
        }
    } else {
        n = cand_compact(s, cs, n, floor_from_max(kmax));
        topk_exact_known = false;
    }
    if (n > SORT_MAX || n < 1) return false;

    // sort by rank counting (all composites distinct)
    if (threadIdx.x < n) {
        const u64 C = cs.cand[threadIdx.x];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += cs.cand[j] > C;
        cs.sorted[rank] = C;
    }
    __syncthreads();

    const int j = threadIdx.x;
    const u64 Cj = j < n ? cs.sorted[j] : 0ull;
    const float zmax = unkey((uint32_t)(cs.sorted[0] >> 32));
    const float zj = unkey((uint32_t)(Cj >> 32));
    const double dj = (double)zj - (double)zmax;
    const int L6 = has_topk ? (n < k ? n : k) : n;

    int n_topk = L6;
    if (!topk_exact_known && a.out_num_topk) {
        // diagnostic only: count the finite scores of the row
        uint32_t local = 0;
        for_each_score<DT>(c, [&](int, float z) { uint32_t kk = key_of(z); local += (kk >= KEY_MIN_FINITE && kk < KEY_POS_INF); });
        u64 nfin = block_sum_u64(s, local);
        n_topk = has_topk ? (int)(nfin < (u64)k ? nfin : (u64)k) : (int)nfin;
    }
    out.n_topk = n_topk;
    if (a.dbg_topk_ids && has_topk && L6 <= a.dbg_cap && j < L6) a.dbg_topk_ids[(int64_t)b * a.dbg_cap + j] = comp_idx(Cj);

    // min-p (a prefix of the order), at least one survivor
    bool in7 = j < L6 && (!has_minp || dj >= ln_minp);
    int L7 = (int)block_sum_u64(s, in7 ? 1u : 0u);
    if (L7 < 1) L7 = 1;
    // top-p over the survivors' mass, fixed-point so that the sums do not depend on the order
    u64 ej = (j < L7) ? __double2ull_rn(exp(dj) * FX50) : 0ull;
    u64 total;
    u64 before = block_exscan_u64(s, ej, total);
    bool keep = j < L7;
    if (!rp.greedy && rp.top_p < 1.0f) {
        double t = ceil((double)rp.top_p * (double)total);
        u64 target = t <= 1.0 ? 1ull : (u64)t;
        if (target > total) target = total;
        keep = keep && before < target;
    }
    const int L8 = (int)block_sum_u64(s, keep ? 1u : 0u);
    const u64 S_fx = block_sum_u64(s, keep ? ej : 0ull);
    const double lnS = log((double)S_fx) - 50.0 * 0.6931471805599453;
    out.n_keep = L8;

    // race
    const int id = comp_idx(Cj);
    u64 G = 0;
    if (keep) {
        double g = dj + neg_log_exp1_f64(race_word(rp.seed, rp.R, a.step, id));
        long long gb = __double_as_longlong(g);
        G = (gb < 0) ? ~(u64)gb : ((u64)gb | 0x8000000000000000ull);
    }
    const u64 Gmax = block_max_u64(s, G);
    const u64 win = block_max_u64(s, (keep && G == Gmax) ? (u64)(uint32_t)(~(uint32_t)id) : 0ull);
    const int tok = (L8 == 1) ? comp_idx(cs.sorted[0]) : (int)(~(uint32_t)win);
    if (keep && id == tok) {
        s.bcast[0] = (u64)__float_as_uint((L8 == 1) ? 0.0f : (float)(dj - lnS));
    }
    __syncthreads();
    out.token = tok;
    out.logprob = __uint_as_float((uint32_t)s.bcast[0]);
    if (a.num_top > 0 && j < a.num_top) {
        const int64_t q = (int64_t)b * a.num_top + j;
        if (j < L8) {
            a.out_top_ids[q] = id;
            a.out_top_logprobs[q] = (L8 == 1) ? 0.0f : (float)(dj - lnS);
        }
    }
    __syncthreads();
    return true;
}

// ------------------------------------------------------------------ the kernel

// dynamic shared memory layout (bytes): [24 KiB shared by the two paths: histograms (cnt 8 KiB, mass
// 16 KiB) or candidates (16 KiB) + sorted list (4 KiB) + 256 bins (1 KiB)][bitmap][coarse][counts]
template <int DT>
__global__ void __launch_bounds__(NT, 2) albireo_sample_kernel(const SampleArgs a) {
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ BlockScratch s;
    const int b = blockIdx.x;
    const int V = a.V;

    HistBins h;
    h.cnt = (uint32_t *)smem;
    h.mass = (u64 *)(smem + HIST_BINS * 4);
    HistSmem hs;
    const int nwords = (V + 31) >> 5, ncoarse = (nwords + 7) >> 3;
    hs.bitmap = (uint32_t *)(smem + HIST_BINS * 12);
    hs.coarse = hs.bitmap + (nwords + 1);
    hs.counts = hs.coarse + (ncoarse + 1);

    RowParams rp;
    rp.T = a.temperature ? a.temperature[b] : 1.0f;
    rp.top_k = a.top_k ? a.top_k[b] : 0;
    rp.top_p = a.top_p ? a.top_p[b] : 1.0f;
    rp.min_p = a.min_p ? a.min_p[b] : 0.0f;
    rp.seed = a.seeds ? a.seeds[b] : 0ull;
    rp.R = a.row_base + (uint32_t)b;
    rp.greedy = !(rp.T > 0.0f);

    RowOut out;
    out.token = 0; out.logprob = 0.0f; out.n_keep = 0; out.n_topk = 0; out.status = 0;
    if (rp.T < 0.0f || rp.T != rp.T) out.status |= ALBIREO_ROW_BAD_PARAM;

    RowCtx c;
    c.row = (const char *)a.logits + (size_t)b * (size_t)a.row_stride * Elem<DT>::SIZE;
    c.V = V;
    c.invT = rp.greedy ? 1.0f : __fdiv_rn(1.0f, rp.T);
    c.r = a.rep ? a.rep[b] : 1.0f;
    c.p = a.pres ? a.pres[b] : 0.0f;
    c.f = a.freq ? a.freq[b] : 0.0f;
    c.has_hist = false; c.bitmap = nullptr; c.coarse = nullptr; c.counts = nullptr;
    if (!(c.r > 0.0f)) out.status |= ALBIREO_ROW_BAD_PARAM;

    if (a.hist_ids && a.hist_off) {
        const int o0 = a.hist_off[b], o1 = a.hist_off[b + 1];
        if (o1 > o0) {
            bool ok = build_history(s, hs, c, a.hist_ids + o0, o1 - o0, a.ws_counts, a.ws_counts_cap, (int64_t)o0);
            c.has_hist = ok;
            if (!ok) out.status |= ALBIREO_ROW_HISTORY_OVERFLOW;
        }
    }

    // dbg / top-N padding first, the paths overwrite what they produce
    if (a.dbg_topk_ids) for (int j = threadIdx.x; j < a.dbg_cap; j += NT) a.dbg_topk_ids[(int64_t)b * a.dbg_cap + j] = -1;
    if (a.num_top > 0) for (int j = threadIdx.x; j < a.num_top; j += NT) {
        a.out_top_ids[(int64_t)b * a.num_top + j] = -1;
        a.out_top_logprobs[(int64_t)b * a.num_top + j] = __uint_as_float(0xFF800000u);
    }
    __syncthreads();

    CandSmem cs;
    cs.cand = (u64 *)smem;                                  // 16 KiB
    cs.sorted = (u64 *)(smem + CAND_CAP * 8);               // 4 KiB
    cs.hist = (uint32_t *)(smem + CAND_CAP * 8 + SORT_MAX * 8);   // 1 KiB
    bool done = false;
    if (!(a.flags & ALBIREO_FLAG_FORCE_GENERAL)) done = candidate_path<DT>(s, cs, c, rp, a, b, out);
    if (!done) {
        __syncthreads();
        general_path<DT>(s, h, c, rp, a, b, out);
    }

    if (threadIdx.x == 0) {
        a.out_tokens[b] = out.token;
        a.out_logprobs[b] = out.logprob;
        if (a.out_num_kept) a.out_num_kept[b] = out.n_keep;
        if (a.out_num_topk) a.out_num_topk[b] = out.n_topk;
        if (a.out_row_status) a.out_row_status[b] = out.status;
    }
}

size_t smem_bytes_for(int V, bool with_history) {
    size_t bytes = (size_t)HIST_BINS * 12;
    if (with_history) {
        size_t nwords = ((size_t)V + 31) / 32, ncoarse = (nwords + 7) / 8;
        bytes += (nwords + 1 + ncoarse + 1 + CNT_CAP) * 4;
    }
    return (bytes + 15) & ~(size_t)15;
}

constexpr size_t WS_HEADER = 256;

}  // namespace

// ------------------------------------------------------------------ C ABI

struct albireo_sampler {
    int32_t device;
    int32_t max_rows, max_vocab;
    int64_t max_history_total;
    unsigned char *workspace;
    size_t workspace_bytes;
    size_t max_smem;
    uint64_t launches;
    char err[256];
};

static void set_err(albireo_sampler *h, const char *fmt, const char *detail) {
    if (h) snprintf(h->err, sizeof h->err, fmt, detail ? detail : "");
}

extern "C" size_t albireo_sample_workspace_bytes(int32_t max_rows, int32_t max_vocab, int64_t max_history_total) {
    if (max_rows < 0 || max_vocab < 0 || max_history_total < 0) return 0;
    size_t bytes = WS_HEADER + (size_t)max_history_total * 4;
    return (bytes + 255) & ~(size_t)255;
}

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

extern "C" size_t albireo_sample_host_staging_bytes(int32_t max_rows, int32_t max_vocab, int64_t max_history_total) {
    if (max_rows < 0 || max_vocab < 0 || max_history_total < 0) return 0;
    size_t B = (size_t)max_rows, V = (size_t)max_vocab, H = (size_t)max_history_total;
    size_t bytes = align256(B * V * 4);                 // logits
    bytes += 7 * align256(B * 4);                       // T, k, top_p, min_p, r, p, f
    bytes += align256(H * 4) + align256((B + 1) * 4);   // history
    bytes += align256(B * 8);                           // seeds
    bytes += 5 * align256(B * 4);                       // tokens, logprobs, num_kept, num_topk, status
    bytes += 2 * align256(B * (size_t)ALBIREO_MAX_NUM_TOP * 4);   // top-N ids, logprobs
    return bytes;
}

extern "C" int albireo_sample_init(albireo_sampler_t **out, int32_t device, int32_t max_rows, int32_t max_vocab,
                                   int64_t max_history_total, void *workspace, size_t workspace_bytes) {
    if (!out) return ALBIREO_EINVAL;
    *out = nullptr;
    if (max_rows < 1 || max_vocab < 1 || max_history_total < 0 || device < 0) return ALBIREO_EINVAL;
    if (max_vocab > ALBIREO_MAX_VOCAB) return ALBIREO_EUNSUPPORTED;
    if (!workspace || ((uintptr_t)workspace & 255u)) return ALBIREO_EINVAL;
    if (workspace_bytes < albireo_sample_workspace_bytes(max_rows, max_vocab, max_history_total)) return ALBIREO_EINVAL;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return ALBIREO_ECUDA;
    if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return ALBIREO_ECUDA; }
    const size_t smem = smem_bytes_for(max_vocab, true);
    cudaError_t e1 = cudaFuncSetAttribute(albireo_sample_kernel<ALBIREO_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    cudaError_t e2 = cudaFuncSetAttribute(albireo_sample_kernel<ALBIREO_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (prev >= 0 && prev != device) cudaSetDevice(prev);
    if (e1 != cudaSuccess || e2 != cudaSuccess) { cudaGetLastError(); return ALBIREO_ECUDA; }

    albireo_sampler *h = new (std::nothrow) albireo_sampler();
    if (!h) return ALBIREO_ENOMEM;
    h->device = device; h->max_rows = max_rows; h->max_vocab = max_vocab;
    h->max_history_total = max_history_total;
    h->workspace = (unsigned char *)workspace; h->workspace_bytes = workspace_bytes;
    h->max_smem = smem; h->launches = 0; h->err[0] = 0;
    *out = h;
    return ALBIREO_OK;
}

extern "C" int albireo_sample(albireo_sampler_t *h, const void *logits, int32_t B, int32_t V, int32_t dtype,
                              const float *temperature, const int32_t *top_k, const float *top_p, const float *min_p,
                              const float *repetition_penalty, const float *presence_penalty,
                              const float *frequency_penalty, const int32_t *history_ids,
                              const int32_t *history_offsets, const uint64_t *seeds, uint64_t step,
                              int32_t *out_tokens, float *out_logprobs, void *stream,
                              const albireo_sample_ext_t *ext) {
    if (!h) return ALBIREO_EINVAL;
    h->err[0] = 0;
    if (B == 0) return ALBIREO_OK;
    if (B < 0 || B > h->max_rows) { set_err(h, "B out of range%s", ""); return ALBIREO_EINVAL; }
    if (V < 1 || V > h->max_vocab) { set_err(h, "V out of range%s", ""); return ALBIREO_EINVAL; }
    if (dtype != ALBIREO_F32 && dtype != ALBIREO_BF16) { set_err(h, "unknown dtype%s", ""); return ALBIREO_EINVAL; }
    if (!logits || !out_tokens || !out_logprobs) { set_err(h, "NULL logits or output%s", ""); return ALBIREO_EINVAL; }
    if ((history_ids == nullptr) != (history_offsets == nullptr)) { set_err(h, "history_ids and history_offsets must both be given%s", ""); return ALBIREO_EINVAL; }
    const size_t esize = dtype == ALBIREO_F32 ? 4 : 2;
    if ((uintptr_t)logits % esize) { set_err(h, "logits not element-aligned%s", ""); return ALBIREO_EINVAL; }

    SampleArgs a;
    memset(&a, 0, sizeof a);
    a.logits = logits; a.B = B; a.V = V; a.row_stride = V;
    a.temperature = temperature; a.top_k = top_k; a.top_p = top_p; a.min_p = min_p;
    a.rep = repetition_penalty; a.pres = presence_penalty; a.freq = frequency_penalty;
    a.hist_ids = history_ids; a.hist_off = history_offsets;
    a.seeds = seeds; a.step = step;
    a.out_tokens = out_tokens; a.out_logprobs = out_logprobs;
    a.ws_counts = (uint32_t *)(h->workspace + WS_HEADER);
    a.ws_counts_cap = h->max_history_total;
    if (ext) {
        if (ext->struct_size != sizeof(albireo_sample_ext_t)) { set_err(h, "ext->struct_size mismatch%s", ""); return ALBIREO_EINVAL; }
        if (ext->row_stride_elems != 0) {
            if (ext->row_stride_elems < V) { set_err(h, "row stride smaller than V%s", ""); return ALBIREO_EINVAL; }
            a.row_stride = ext->row_stride_elems;
        }
        a.row_base = ext->row_base; a.flags = ext->flags;
        if (ext->num_top < 0 || ext->num_top > ALBIREO_MAX_NUM_TOP) { set_err(h, "num_top out of range%s", ""); return ALBIREO_EUNSUPPORTED; }
        if (ext->num_top > 0 && (!ext->out_top_ids || !ext->out_top_logprobs)) { set_err(h, "num_top > 0 needs both top-N outputs%s", ""); return ALBIREO_EINVAL; }
        a.num_top = ext->num_top; a.out_top_ids = ext->out_top_ids; a.out_top_logprobs = ext->out_top_logprobs;
        a.out_num_kept = ext->out_num_kept; a.out_num_topk = ext->out_num_topk;
        if (ext->dbg_cap < 0 || (ext->dbg_cap > 0 && !ext->dbg_topk_ids)) { set_err(h, "bad dbg_cap / dbg_topk_ids%s", ""); return ALBIREO_EINVAL; }
        a.dbg_cap = ext->dbg_topk_ids ? ext->dbg_cap : 0;
        a.dbg_topk_ids = ext->dbg_cap > 0 ? ext->dbg_topk_ids : nullptr;
        a.out_row_status = ext->out_row_status;
    }
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess || cur != h->device) { cudaGetLastError(); set_err(h, "the handle's device is not current%s", ""); return ALBIREO_EINVAL; }

    const size_t smem = smem_bytes_for(V, history_ids != nullptr);
    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == ALBIREO_F32) albireo_sample_kernel<ALBIREO_F32><<<B, NT, smem, st>>>(a);
    else albireo_sample_kernel<ALBIREO_BF16><<<B, NT, smem, st>>>(a);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_err(h, "kernel launch failed: %s", cudaGetErrorString(e)); return ALBIREO_ECUDA; }
    h->launches += 1;
    return ALBIREO_OK;
}

extern "C" int albireo_sample_host(albireo_sampler_t *h, const void *logits, int32_t B, int32_t V, int32_t dtype,
                                   const float *temperature, const int32_t *top_k, const float *top_p,
                                   const float *min_p, const float *repetition_penalty,
                                   const float *presence_penalty, const float *frequency_penalty,
                                   const int32_t *history_ids, const int32_t *history_offsets, int64_t history_total,
                                   const uint64_t *seeds, uint64_t step, int32_t *out_tokens, float *out_logprobs,
                                   void *stream, const albireo_sample_ext_t *ext) {
    if (!h) return ALBIREO_EINVAL;
    h->err[0] = 0;
    if (B == 0) return ALBIREO_OK;
    if (B < 0 || B > h->max_rows || V < 1 || V > h->max_vocab) { set_err(h, "B or V out of range%s", ""); return ALBIREO_EINVAL; }
    if (dtype != ALBIREO_F32 && dtype != ALBIREO_BF16) { set_err(h, "unknown dtype%s", ""); return ALBIREO_EINVAL; }
    if (!logits || !out_tokens || !out_logprobs) { set_err(h, "NULL logits or output%s", ""); return ALBIREO_EINVAL; }
    if ((history_ids == nullptr) != (history_offsets == nullptr) || history_total < 0 || history_total > h->max_history_total) {
        set_err(h, "bad history arguments%s", ""); return ALBIREO_EINVAL;
    }
    if (ext && ext->struct_size != sizeof(albireo_sample_ext_t)) { set_err(h, "ext->struct_size mismatch%s", ""); return ALBIREO_EINVAL; }
    if (ext && ext->row_stride_elems != 0 && ext->row_stride_elems != V) { set_err(h, "host entry needs dense rows%s", ""); return ALBIREO_EINVAL; }
    if (ext && ext->dbg_cap > 0) { set_err(h, "host entry has no debug output%s", ""); return ALBIREO_EINVAL; }
    const size_t base = albireo_sample_workspace_bytes(h->max_rows, h->max_vocab, h->max_history_total);
    if (h->workspace_bytes < base + albireo_sample_host_staging_bytes(h->max_rows, h->max_vocab, h->max_history_total)) {
        set_err(h, "workspace given to init has no staging space%s", ""); return ALBIREO_EINVAL;
    }
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess || cur != h->device) { cudaGetLastError(); set_err(h, "the handle's device is not current%s", ""); return ALBIREO_EINVAL; }

    cudaStream_t st = (cudaStream_t)stream;
    unsigned char *p = h->workspace + base;
    cudaError_t e = cudaSuccess;
    auto stage = [&](const void *src, size_t bytes) -> void * {
        void *dst = p;
        p += align256(bytes);
        if (src && bytes && e == cudaSuccess) e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, st);
        return src ? dst : nullptr;
    };
    auto reserve = [&](size_t bytes) -> void * { void *dst = p; p += align256(bytes); return dst; };
    const size_t Bs = (size_t)B, esize = dtype == ALBIREO_F32 ? 4 : 2;
    const void *d_logits = stage(logits, Bs * (size_t)V * esize);
    const float *d_T = (const float *)stage(temperature, Bs * 4);
    const int32_t *d_k = (const int32_t *)stage(top_k, Bs * 4);
    const float *d_tp = (const float *)stage(top_p, Bs * 4);
    const float *d_mp = (const float *)stage(min_p, Bs * 4);
    const float *d_r = (const float *)stage(repetition_penalty, Bs * 4);
    const float *d_p = (const float *)stage(presence_penalty, Bs * 4);
    const float *d_f = (const float *)stage(frequency_penalty, Bs * 4);
    const int32_t *d_hid = (const int32_t *)stage(history_ids, (size_t)history_total * 4);
    const int32_t *d_hoff = (const int32_t *)stage(history_offsets, (Bs + 1) * 4);
    const uint64_t *d_seeds = (const uint64_t *)stage(seeds, Bs * 8);
    int32_t *d_tok = (int32_t *)reserve(Bs * 4);
    float *d_lp = (float *)reserve(Bs * 4);
    albireo_sample_ext_t dx;
    memset(&dx, 0, sizeof dx);
    dx.struct_size = sizeof dx;
    if (ext) {
        dx.flags = ext->flags; dx.row_base = ext->row_base; dx.num_top = ext->num_top;
        if (ext->num_top < 0 || ext->num_top > ALBIREO_MAX_NUM_TOP) { set_err(h, "num_top out of range%s", ""); return ALBIREO_EUNSUPPORTED; }
        if (ext->out_num_kept) dx.out_num_kept = (int32_t *)reserve(Bs * 4);
        if (ext->out_num_topk) dx.out_num_topk = (int32_t *)reserve(Bs * 4);
        if (ext->out_row_status) dx.out_row_status = (uint32_t *)reserve(Bs * 4);
        if (ext->num_top > 0) {
            dx.out_top_ids = (int32_t *)reserve(Bs * (size_t)ext->num_top * 4);
            dx.out_top_logprobs = (float *)reserve(Bs * (size_t)ext->num_top * 4);
        }
    }
    if (e != cudaSuccess) { set_err(h, "host-to-device copy failed: %s", cudaGetErrorString(e)); cudaGetLastError(); return ALBIREO_ECUDA; }
    int rc = albireo_sample(h, d_logits, B, V, dtype, d_T, d_k, d_tp, d_mp, d_r, d_p, d_f, d_hid, d_hoff, d_seeds, step,
                            d_tok, d_lp, stream, &dx);
    if (rc != ALBIREO_OK) return rc;
    auto back = [&](void *dst, const void *src, size_t bytes) {
        if (dst && src && e == cudaSuccess) e = cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, st);
    };
    back(out_tokens, d_tok, Bs * 4);
    back(out_logprobs, d_lp, Bs * 4);
    if (ext) {
        back(ext->out_num_kept, dx.out_num_kept, Bs * 4);
        back(ext->out_num_topk, dx.out_num_topk, Bs * 4);
        back(ext->out_row_status, dx.out_row_status, Bs * 4);
        if (ext->num_top > 0) {
            back(ext->out_top_ids, dx.out_top_ids, Bs * (size_t)ext->num_top * 4);
            back(ext->out_top_logprobs, dx.out_top_logprobs, Bs * (size_t)ext->num_top * 4);
        }
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) { set_err(h, "copy back / synchronize failed: %s", cudaGetErrorString(e)); return ALBIREO_ECUDA; }
    return ALBIREO_OK;
}

extern "C" int albireo_sample_destroy(albireo_sampler_t *h) {
    delete h;
    return ALBIREO_OK;
}

extern "C" const char *albireo_last_error(const albireo_sampler_t *h) { return h ? h->err : ""; }

extern "C" uint64_t albireo_sample_launch_count(const albireo_sampler_t *h) { return h ? h->launches : 0; }
