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

#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>
#include <mutex>
#include <new>

#include "albireo_sample.h"

namespace cg = cooperative_groups;

namespace {

typedef unsigned long long u64;

constexpr int NT = 512;                 // threads per CTA
constexpr int NWARPS = NT / 32;
constexpr int HIST_BINS = 2048;         // 11-bit digits
constexpr int CNT_CAP = 2048;           // on-chip slots for distinct history ids per row
constexpr int CAND_CAP = 1024;          // candidate buffer entries (candidate path)
constexpr int SORT_MAX = 512;           // most candidates the final stage sorts (== NT)
constexpr int KA_MAX = 256;             // largest top-k the candidate path takes
constexpr int TILE_VECS = 4;            // 16-byte vectors per thread per tile
constexpr int STAGE_BYTES = NT * TILE_VECS * 16;   // one ring stage = one tile (32 KiB)
constexpr int MAX_STAGES = 8;
constexpr int WAIT_CAP = 1 << 20;       // mbarrier polls before a wait gives up
constexpr int COMMON_BYTES = 10240;     // candidate composites (8 KiB) + select bins (2 KiB)
constexpr uint32_t KEY_MIN_FINITE = 0x00800000u;   // key(-FLT_MAX); key(-inf) is one below
constexpr uint32_t KEY_POS_INF = 0xFF800000u;      // key(+inf)
constexpr float FX_SCALE = 1099511627776.0f;       // 2^40: fixed-point scale of masses
constexpr double LN2_40 = 27.725887222397812;      // 40 ln 2

struct SampleArgs {
    // (ordered by first use: a launch's arguments sit in constant memory no SM has seen before, and
    // every 64-byte line of them costs a miss at first touch)
    const void *logits;
    int32_t B, V;
    int64_t row_stride;
    int32_t nseg;               // pieces per row (1: rows are contiguous)
    int32_t nstages;            // ring depth chosen by the host for this launch
    int32_t vps;                // 16-byte vectors per piece (worked out on the host: no division on the device)
    int32_t Vs;                 // elements per piece
    uint32_t flags;
    uint32_t row_base;
    const float *temperature;
    const int32_t *top_k;
    const float *top_p, *min_p, *rep, *pres, *freq;
    const int32_t *hist_ids, *hist_off;
    const uint64_t *seeds;
    const int32_t *out_start;   // per row: where the generated output begins in the history, or null: at 0
    uint64_t step;
    int32_t *out_tokens;
    float *out_logprobs;
    int32_t num_top;
    int32_t dbg_cap;
    int32_t *out_top_ids;
    float *out_top_logprobs;
    int32_t *out_num_kept, *out_num_topk;
    int32_t *dbg_topk_ids;
    uint32_t *out_row_status;
    const float *exp1;          // pre-generated Exp(1) variates [B, exp1_stride], or null: counter-based draw
    int64_t exp1_stride;
    int32_t *backfill_ids;      // early feedback: next iteration's input ids, or null
    const int32_t *backfill_index;
    int64_t backfill_len;
    unsigned long long *feedback_ring;   // (row id << 32 | token) records for the output processor, or null
    int64_t feedback_cap, feedback_head;
    uint32_t *ws_counts;        // global scratch for history counts of rows with many distinct ids
    int64_t ws_counts_cap;      // entries
    int32_t elem_size;          // host side only: bytes per logit
    // rows in pieces (vocabulary shards as the all-to-all of sequence-parallel sampling leaves them)
    int32_t seg_ptr_count;      // > 0: the pieces live in buffers of their own, seg_ptr[j]; 0: a stride apart in `logits`
    int64_t seg_stride;         // elements between consecutive pieces of a row
    int64_t seg_row_offset;     // rows to skip at the start of every piece buffer
    const void *seg_ptr[ALBIREO_MAX_PEER_SEGMENTS];
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
// The same quantity for the general path, where it is evaluated once per kept element of rows that
// may keep tens of thousands: branch-free, hardware logarithms.  E = v + v^2/2 + ... for v < 1/4
// (the small-E end decides the race and keeps full relative accuracy there), E = -ln(1 - v) above;
// absolute error of the result about 1e-6, inside the band in which the race counts as a near-tie.
__device__ __forceinline__ float neg_log_exp1_fast(uint32_t w) {
    const float v = __fmaf_rn((float)w, 2.3283064365386963e-10f, 1.1641532182693481e-10f);
    float p = 1.0f / 12.0f;
#pragma unroll
    for (int n = 11; n >= 1; --n) p = __fmaf_rn(p, v, 1.0f / (float)n);
    const float e_small = p * v;
    const float omv = __fmaf_rn((float)(~w), 2.3283064365386963e-10f, 1.1641532182693481e-10f);
    const float e_large = -__logf(omv);
    const float E = v < 0.25f ? e_small : e_large;
    return -__logf(E);
}

__device__ __forceinline__ uint32_t orderable_f32(float g) { return key_of(g); }

// fixed-point mass of an element at distance d = z - zmax <= 0 (deterministic integer sums)
__device__ __forceinline__ u64 mass_fx(float d) {
    return __float2ull_rn(expf(d) * FX_SCALE);
}

// ------------------------------------------------------------------ block primitives

// what the general path needs of the launch arguments (see general_path_call)
struct GenArgs {
    int32_t *dbg_topk_ids; const float *exp1; int64_t exp1_stride; int32_t *out_top_ids; float *out_top_logprobs;
    uint64_t step; uint32_t flags; int32_t num_top; int32_t dbg_cap;
};

struct BlockScratch {
    u64 red[NWARPS];
    u64 red2[NWARPS];
    u64 bcast[4];
    uint32_t found_digit, found_cnt;
    u64 found_above;
    uint32_t list_cnt;
    uint32_t cand_cnt, overflow, runmax, timeout;
    uint32_t r32a[NWARPS], r32b[NWARPS];
    uint32_t mm_max, mm_min;
    uint32_t done[MAX_STAGES];   // warps finished with each ring stage
    uint32_t maint_at;           // tile index before which every warp meets (0xFFFFFFFF: none)
    uint32_t issued;             // tiles whose copy has been issued so far
    const char *seg_base[ALBIREO_MAX_SEGMENTS];   // where this row's pieces start (rows in pieces only)
    uint32_t nfin_cap;           // general path: min(#finite scores, ALBIREO_MAX_NUM_TOP + 1), parked here until the list is written
    GenArgs ga;                  // the general path's copy of the launch arguments it uses
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
    // a row may arrive as nseg equal pieces of Vs elements (vocabulary shards as the all-to-all of
    // sequence-parallel sampling leaves them, section 6.1 step 2), in one buffer a stride apart or in a
    // buffer each (other workers' memory included); nseg == 1: one piece
    int nseg, Vs;
    const char *const *seg_base;   // shared-memory table: start of each piece of this row
    float invT, r, p, f;
    bool has_hist;
    const uint32_t *bitmap;   // V bits (+1 pad word): token appears in the history
    const uint32_t *coarse;   // exclusive popcount prefix per 8 bitmap words
    const uint32_t *counts;   // occurrence count per distinct id, indexed by rank in the bitmap
    uint32_t n_distinct;      // number of distinct history ids (set bits of the bitmap)
    int ncoarse;              // entries of `coarse`
};

__device__ __forceinline__ uint32_t hist_rank(const RowCtx &c, int i) {
    int w = i >> 5, cb = w >> 3;
    uint32_t r = c.coarse[cb];
    for (int ww = cb << 3; ww < w; ++ww) r += __popc(c.bitmap[ww]);
    r += __popc(c.bitmap[w] & ((1u << (i & 31)) - 1u));
    return r;
}

// penalties: each line is one rounded fp32 operation
// the penalties of a token seen in the history, `cnt` of its occurrences in the generated output
// (all of them when the history is not split; 0 for a token seen in the prompt only)
__device__ __forceinline__ float penalise_counted(const RowCtx &c, float x, uint32_t cnt) {
    float a = (x > 0.0f) ? __fdiv_rn(x, c.r) : __fmul_rn(x, c.r);
    a = __fsub_rn(a, __fmul_rn(c.f, __uint2float_rn(cnt)));
    if (cnt) a = __fsub_rn(a, c.p);
    return a;
}
__device__ __forceinline__ float penalise(const RowCtx &c, int i, float x) {
    return penalise_counted(c, x, c.counts[hist_rank(c, i)]);
}

template <int DT> struct Elem;
template <> struct Elem<ALBIREO_F32> {
    static constexpr int SIZE = 4, PER_VEC = 4;
    static __device__ __forceinline__ float load(const void *row, int i) { return __ldg((const float *)row + i); }
    // plain load through a generic pointer (shared memory allowed)
    static __device__ __forceinline__ float load_plain(const void *p, int i) { return ((const float *)p)[i]; }
    static __device__ __forceinline__ float get(const uint4 &q, int e) {
        return __uint_as_float(e == 0 ? q.x : e == 1 ? q.y : e == 2 ? q.z : q.w);
    }
};
template <> struct Elem<ALBIREO_BF16> {
    static constexpr int SIZE = 2, PER_VEC = 8;
    static __device__ __forceinline__ float load(const void *row, int i) {
        return __uint_as_float(((uint32_t)__ldg((const unsigned short *)row + i)) << 16);
    }
    static __device__ __forceinline__ float load_plain(const void *p, int i) {
        return __uint_as_float(((uint32_t)((const unsigned short *)p)[i]) << 16);
    }
    static __device__ __forceinline__ float get(const uint4 &q, int e) {
        uint32_t w = (e >> 1) == 0 ? q.x : (e >> 1) == 1 ? q.y : (e >> 1) == 2 ? q.z : q.w;
        return __uint_as_float((e & 1) ? (w & 0xFFFF0000u) : (w << 16));
    }
};

template <> struct Elem<ALBIREO_F16> {
    static constexpr int SIZE = 2, PER_VEC = 8;
    static __device__ __forceinline__ float load(const void *row, int i) {
        return __half2float(__ushort_as_half(__ldg((const unsigned short *)row + i)));
    }
    static __device__ __forceinline__ float load_plain(const void *p, int i) {
        return __half2float(__ushort_as_half(((const unsigned short *)p)[i]));
    }
    static __device__ __forceinline__ float get(const uint4 &q, int e) {
        uint32_t w = (e >> 1) == 0 ? q.x : (e >> 1) == 1 ? q.y : (e >> 1) == 2 ? q.z : q.w;
        return __half2float(__ushort_as_half((unsigned short)((e & 1) ? (w >> 16) : (w & 0xFFFFu))));
    }
};

// address of element i of the row
template <int DT>
__device__ __forceinline__ const void *elem_ptr(const RowCtx &c, int i) {
    if (c.nseg == 1) return (const char *)c.row + (size_t)i * Elem<DT>::SIZE;
    const int j = i / c.Vs;
    return c.seg_base[j] + (size_t)(i - j * c.Vs) * Elem<DT>::SIZE;
}
// address of the row's v-th 16-byte vector (rows in pieces are 16-byte aligned piece by piece, so
// their vectors start at element 0 and none straddles two pieces)
template <int DT>
__device__ __forceinline__ const uint4 *vec_ptr(const RowCtx &c, const uint4 *vp, int v) {
    if (c.nseg == 1) return vp + v;
    const int vps = c.Vs / Elem<DT>::PER_VEC;
    const int j = v / vps;
    return (const uint4 *)c.seg_base[j] + (v - j * vps);
}

__device__ __forceinline__ float score_of(const RowCtx &c, int i, float x) {
    float a = x;
    if (c.has_hist && ((c.bitmap[i >> 5] >> (i & 31)) & 1u)) a = penalise(c, i, x);
    return __fmul_rn(a, c.invT);
}

__device__ int hist_id_of_rank(const RowCtx &c, uint32_t r);

// Vector pre-test per dtype, in the domain the test runs in.
// 16-bit types: raw logits; the threshold is the smallest raw value whose score has key >= tau
// (packed twice).  x -> fl32(x * invT) is increasing, strictly so on distinct 16-bit values unless
// the product leaves the fp32 range, so a compare of raw values is a superset of the key test.
// fp32: scores; the threshold is unkey(tau).
struct Bf16Packed {
    typedef __nv_bfloat162 H2;
    static constexpr uint32_t LO = 0x0080u, HI = 0xFF7Fu, NEG_INF = 0xFF80u;    // order codes of the finite range; -inf pattern
    static __device__ __forceinline__ float widen(uint32_t bits) { return __uint_as_float(bits << 16); }
    static __device__ __forceinline__ uint32_t truncate(float x) { return __float_as_uint(x) >> 16; }
};
struct F16Packed {
    typedef __half2 H2;
    static constexpr uint32_t LO = 0x0400u, HI = 0xFBFFu, NEG_INF = 0xFC00u;
    static __device__ __forceinline__ float widen(uint32_t bits) { return __half2float(__ushort_as_half((unsigned short)bits)); }
    static __device__ __forceinline__ uint32_t truncate(float x) { return __half_as_ushort(__float2half_rz(x)); }
};
template <int DT> struct VecTest;
template <class P> struct VecTest16 {
    typedef typename P::H2 H2;
    static __device__ uint32_t raw_threshold(uint32_t tau_key, float invT) {
        // order code of a 16-bit pattern (the analogue of the score key) and back
        auto bits_of = [](uint32_t kk) { return (kk & 0x8000u) ? (kk & 0x7FFFu) : (~kk & 0xFFFFu); };
        auto passes = [&](uint32_t kk) {
            float x = P::widen(bits_of(kk));
            return key_of(__fmul_rn(x, invT)) >= tau_key;
        };
        constexpr uint32_t LO = P::LO, HI = P::HI;             // the finite codes
        // a guess from an approximate quotient, truncated to 16 bits: the answer is the guess or a
        // neighbour, so the four codes around it are tried at once instead of one after another
        const float xg = __fdividef(unkey(tau_key), invT);
        const uint32_t b16 = P::truncate(xg) & 0xFFFFu;
        uint32_t k16 = (b16 & 0x8000u) ? (~b16 & 0xFFFFu) : (b16 | 0x8000u);
        k16 = k16 < LO + 2u ? LO + 2u : (k16 > HI - 1u ? HI - 1u : k16);
        const bool p0 = passes(k16 - 2u), p1 = passes(k16 - 1u), p2 = passes(k16), p3 = passes(k16 + 1u);
        uint32_t ans = 0;
        if (p1 && !p0) ans = k16 - 1u;
        else if (p2 && !p1) ans = k16;
        else if (p3 && !p2) ans = k16 + 1u;
        if (ans == 0) {
            // not bracketed (an extreme temperature, or the ends of the range): a short walk
            int it = 0;
            while (it < 16 && k16 > LO && passes(k16)) { --k16; ++it; }
            while (it < 32 && k16 < HI && !passes(k16)) { ++k16; ++it; }
            const bool ok = passes(k16) && (k16 == LO || !passes(k16 - 1u));
            ans = ok ? k16 : 0u;
        }
        const uint32_t b = ans ? bits_of(ans) : P::NEG_INF;    // not settled: let everything through
        return b | (b << 16);
    }
    static __device__ __forceinline__ H2 vmax(const uint4 &q) {
        H2 a = __hmax2(*reinterpret_cast<const H2 *>(&q.x), *reinterpret_cast<const H2 *>(&q.y));
        H2 b2 = __hmax2(*reinterpret_cast<const H2 *>(&q.z), *reinterpret_cast<const H2 *>(&q.w));
        return __hmax2(a, b2);
    }
    static __device__ __forceinline__ bool may_pass(const uint4 &q, uint32_t thr, float) {
        return __hge2_mask(vmax(q), *reinterpret_cast<const H2 *>(&thr)) != 0u;
    }
    static __device__ __forceinline__ bool any_may_pass(const uint4 (&q)[TILE_VECS], uint32_t thr, float) {
        H2 m = vmax(q[0]);
#pragma unroll
        for (int u = 1; u < TILE_VECS; ++u) m = __hmax2(m, vmax(q[u]));
        return __hge2_mask(m, *reinterpret_cast<const H2 *>(&thr)) != 0u;
    }
    // bit e set: raw element e >= the raw threshold (a superset of "score key >= tau")
    static __device__ __forceinline__ uint32_t elem_bits(const uint4 &q, uint32_t thr, float) {
        const H2 t2 = *reinterpret_cast<const H2 *>(&thr);
        const uint32_t r0 = __hge2_mask(*reinterpret_cast<const H2 *>(&q.x), t2);
        const uint32_t r1 = __hge2_mask(*reinterpret_cast<const H2 *>(&q.y), t2);
        const uint32_t r2 = __hge2_mask(*reinterpret_cast<const H2 *>(&q.z), t2);
        const uint32_t r3 = __hge2_mask(*reinterpret_cast<const H2 *>(&q.w), t2);
        return ((r0 & 1u) | ((r0 >> 15) & 2u)) | (((r1 & 1u) | ((r1 >> 15) & 2u)) << 2) |
               (((r2 & 1u) | ((r2 >> 15) & 2u)) << 4) | (((r3 & 1u) | ((r3 >> 15) & 2u)) << 6);
    }
    // key of the score of the vector's largest element (an element of the row)
    static __device__ __forceinline__ uint32_t vmax_key(const uint4 &q, float invT) {
        H2 m = vmax(q);
        return key_of(__fmul_rn(fmaxf(__low2float(m), __high2float(m)), invT));
    }
    static __device__ __forceinline__ uint4 fill() { const uint32_t f = P::NEG_INF | (P::NEG_INF << 16); return make_uint4(f, f, f, f); }
    // the raw threshold that only +inf reaches (NEG_INF without its sign bit), packed twice
    static __device__ __forceinline__ uint32_t pos_inf_threshold() { const uint32_t b = P::NEG_INF & 0x7FFFu; return b | (b << 16); }
    // how many of the vector's elements are -inf
    static __device__ __forceinline__ uint32_t count_neginf(const uint4 &q) {
        const uint32_t f = P::NEG_INF | (P::NEG_INF << 16);
        const H2 ninf = *reinterpret_cast<const H2 *>(&f);
        const uint32_t r0 = __heq2_mask(*reinterpret_cast<const H2 *>(&q.x), ninf), r1 = __heq2_mask(*reinterpret_cast<const H2 *>(&q.y), ninf);
        const uint32_t r2 = __heq2_mask(*reinterpret_cast<const H2 *>(&q.z), ninf), r3 = __heq2_mask(*reinterpret_cast<const H2 *>(&q.w), ninf);
        if (!(r0 | r1 | r2 | r3)) return 0u;
        return (uint32_t)(__popc(r0) + __popc(r1) + __popc(r2) + __popc(r3)) >> 4;
    }
};
template <> struct VecTest<ALBIREO_BF16> : VecTest16<Bf16Packed> {};
template <> struct VecTest<ALBIREO_F16> : VecTest16<F16Packed> {};
template <> struct VecTest<ALBIREO_F32> {
    static __device__ uint32_t raw_threshold(uint32_t tau_key, float) { return __float_as_uint(unkey(tau_key)); }
    static __device__ __forceinline__ float vmaxz(const uint4 &q, float invT) {
        return fmaxf(fmaxf(__fmul_rn(__uint_as_float(q.x), invT), __fmul_rn(__uint_as_float(q.y), invT)),
                     fmaxf(__fmul_rn(__uint_as_float(q.z), invT), __fmul_rn(__uint_as_float(q.w), invT)));
    }
    static __device__ __forceinline__ bool may_pass(const uint4 &q, uint32_t thr, float invT) {
        return vmaxz(q, invT) >= __uint_as_float(thr);
    }
    static __device__ __forceinline__ bool any_may_pass(const uint4 (&q)[TILE_VECS], uint32_t thr, float invT) {
        float m = vmaxz(q[0], invT);
#pragma unroll
        for (int u = 1; u < TILE_VECS; ++u) m = fmaxf(m, vmaxz(q[u], invT));
        return m >= __uint_as_float(thr);
    }
    static __device__ __forceinline__ uint32_t elem_bits(const uint4 &q, uint32_t thr, float invT) {
        const float t = __uint_as_float(thr);
        return (uint32_t)(__fmul_rn(__uint_as_float(q.x), invT) >= t) | ((uint32_t)(__fmul_rn(__uint_as_float(q.y), invT) >= t) << 1) |
               ((uint32_t)(__fmul_rn(__uint_as_float(q.z), invT) >= t) << 2) | ((uint32_t)(__fmul_rn(__uint_as_float(q.w), invT) >= t) << 3);
    }
    static __device__ __forceinline__ uint32_t vmax_key(const uint4 &q, float invT) { return key_of(vmaxz(q, invT)); }
    static __device__ __forceinline__ uint4 fill() { return make_uint4(0xFF800000u, 0xFF800000u, 0xFF800000u, 0xFF800000u); }
    static __device__ __forceinline__ uint32_t pos_inf_threshold() { return 0x7F800000u; }
    static __device__ __forceinline__ uint32_t count_neginf(const uint4 &q) {
        return (uint32_t)(q.x == 0xFF800000u) + (uint32_t)(q.y == 0xFF800000u) + (uint32_t)(q.z == 0xFF800000u) + (uint32_t)(q.w == 0xFF800000u);
    }
};

// The part of a row the vector loop does not cover: the scalar head and tail of a row that is not
// 16-byte aligned / not a whole number of vectors, and the penalised tokens from the history tables.
template <int DT, class F>
__device__ __forceinline__ void for_each_score_rest(const RowCtx &c, int head, int nvec, F &&fn) {
    typedef Elem<DT> E;
    const int V = c.V;
    const int tail0 = head + nvec * E::PER_VEC;
    for (int q = threadIdx.x; q < head + (V - tail0); q += NT) {
        const int i = q < head ? q : tail0 + (q - head);
        if (c.has_hist && ((c.bitmap[i >> 5] >> (i & 31)) & 1u)) continue;
        fn(i, __fmul_rn(E::load(elem_ptr<DT>(c, i), 0), c.invT));
    }
    if (c.has_hist) {
        for (uint32_t r = threadIdx.x; r < c.n_distinct; r += NT) {
            const int i = hist_id_of_rank(c, r);
            const float x = E::load(elem_ptr<DT>(c, i), 0);
            const float av = penalise_counted(c, x, c.counts[r]);
            fn(i, __fmul_rn(av, c.invT));
        }
    }
}

// Calls fn(i, z_i) exactly once for every element of the row (each thread a share; any order).
// Unpenalised elements come from 16-byte vector loads over the aligned middle of the row, two
// loads in flight per thread, plus a scalar head and tail; penalised tokens (whose raw value is not
// their score) are skipped there and taken from the history tables afterwards.
template <int DT, class F>
__device__ __forceinline__ void for_each_score(const RowCtx &c, F &&fn) {
    typedef Elem<DT> E;
    const int V = c.V;
    const uintptr_t addr = (uintptr_t)c.row;
    int head = (int)(((16u - (uint32_t)(addr & 15u)) & 15u) / E::SIZE);
    if (head > V) head = V;
    const int nvec = (V - head) / E::PER_VEC;
    const uint4 *vp = (const uint4 *)((const char *)c.row + (size_t)head * E::SIZE);
    for (int v0 = threadIdx.x; v0 < nvec; v0 += 2 * NT) {
        const int v1 = v0 + NT;
        const uint4 q0 = __ldg(vec_ptr<DT>(c, vp, v0));
        const uint4 q1 = v1 < nvec ? __ldg(vec_ptr<DT>(c, vp, v1)) : q0;
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (u == 1 && v1 >= nvec) break;
            const uint4 &q = u ? q1 : q0;
            const int i0 = head + (u ? v1 : v0) * E::PER_VEC;
            uint32_t m = 0;
            if (c.has_hist) m = __funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31);
#pragma unroll
            for (int e = 0; e < E::PER_VEC; ++e)
                if (!((m >> e) & 1u)) fn(i0 + e, __fmul_rn(E::get(q, e), c.invT));
        }
    }
    for_each_score_rest<DT>(c, head, nvec, fn);
}

// Pass 0 of the general path: the largest score key of the row and how many scores are finite.
// Vectors without penalised tokens go through the packed maximum of the candidate path (the map
// from raw value to score is increasing) with four loads in flight; the others element by element.
template <int DT>
__device__ __forceinline__ void pass0_max_count(const RowCtx &c, uint32_t &kbest, uint32_t &nfin) {
    typedef Elem<DT> E;
    typedef VecTest<DT> T;
    const int V = c.V;
    const uintptr_t addr = (uintptr_t)c.row;
    int head = (int)(((16u - (uint32_t)(addr & 15u)) & 15u) / E::SIZE);
    if (head > V) head = V;
    const int nvec = (V - head) / E::PER_VEC;
    const uint4 *vp = (const uint4 *)((const char *)c.row + (size_t)head * E::SIZE);
    auto one = [&](int, float z) {
        const uint32_t k = key_of(z);
        kbest = k > kbest ? k : kbest;
        nfin += (k >= KEY_MIN_FINITE && k < KEY_POS_INF);
    };
    for (int v0 = threadIdx.x; v0 < nvec; v0 += 4 * NT) {
        uint4 q[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) q[u] = (v0 + u * NT < nvec) ? __ldg(vec_ptr<DT>(c, vp, v0 + u * NT)) : T::fill();
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int v = v0 + u * NT;
            if (v >= nvec) break;
            const int i0 = head + v * E::PER_VEC;
            uint32_t m = 0;
            if (c.has_hist) m = __funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31) & ((1u << E::PER_VEC) - 1u);
            if (m == 0) {
                const uint32_t k = T::vmax_key(q[u], c.invT);
                kbest = k > kbest ? k : kbest;
                nfin += (uint32_t)E::PER_VEC - T::count_neginf(q[u]);
            } else {
#pragma unroll
                for (int e = 0; e < E::PER_VEC; ++e)
                    if (!((m >> e) & 1u)) one(i0 + e, __fmul_rn(E::get(q[u], e), c.invT));
            }
        }
    }
    for_each_score_rest<DT>(c, head, nvec, one);
}

// ------------------------------------------------------------------ history -> bitmap + counts

struct HistSmem {
    uint32_t *bitmap;   // nwords + 1
    uint32_t *coarse;   // ncoarse + 1
    uint32_t *counts;   // CNT_CAP
};

// exclusive prefix sum of 32-bit values over the threads of the block (thread order); block total in `total`
__device__ uint32_t block_exscan_u32(BlockScratch &s, uint32_t v, uint32_t &total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, o); if (lane >= o) inc += t; }
    __syncthreads();
    if (lane == 31) s.r32b[wid] = inc;
    __syncthreads();
    uint32_t base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < NWARPS; ++w) { const uint32_t t = s.r32b[w]; base += (w < wid) ? t : 0u; tot += t; }
    total = tot;
    return base + inc - v;
}

// The first HIST_STAGED ids of a row's history are copied into shared memory at the very start of the
// row (asynchronous 4-byte copies, no registers held, by the threads after warp 0, which is busy
// starting the ring): the two sweeps over the ids then read them from there.  What is left of a
// longer history is re-read from global memory.  The staging area is the candidate list, which
// nothing uses before the stream begins.
constexpr int HIST_STAGED = CAND_CAP * 2;      // 8 KiB of ids
constexpr int HIST_HOLDERS = NT - 32;
__device__ __forceinline__ void hist_prefetch(const int32_t *ids, int len, int32_t *staged) {
    if (threadIdx.x < 32) return;
    const int n = len < HIST_STAGED ? len : HIST_STAGED;
    for (int j = (int)threadIdx.x - 32; j < n; j += HIST_HOLDERS)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(staged + j)), "l"(ids + j) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
}

// Builds the per-row penalty tables from the staged ids (see hist_prefetch) and, for a longer
// history, the rest of `ids`.  Returns false (penalties skipped) if the distinct ids fit neither on
// chip nor in the caller's workspace.
// Ids before position out_start are the prompt: they set their bit (repetition penalty) but are not counted.
// Histories repeat a few ids very often: a bit already set is not set again.  (Combining equal ids
// within a warp first, with match.any, was measured and cost far more than the atomics it saved.)
__device__ bool build_history(BlockScratch &s, const HistSmem &hs, RowCtx &c, const int32_t *ids, int len, int out_start,
                              const int32_t *staged, uint32_t *ws, int64_t ws_cap, int64_t ws_off) {
    const int V = c.V;
    const int nwords = (V + 31) >> 5, ncoarse = (nwords + 7) >> 3;
    const int nst = len < HIST_STAGED ? len : HIST_STAGED;
    for (int w = threadIdx.x; w <= nwords; w += NT) hs.bitmap[w] = 0;
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    for (int j = threadIdx.x; j < nst; j += NT) {
        const int t = staged[j];
        if (t >= 0 && t < V) {
            const uint32_t bit = 1u << (t & 31);
            if (!(*(volatile uint32_t *)&hs.bitmap[t >> 5] & bit)) atomicOr(&hs.bitmap[t >> 5], bit);
        }
    }
    for (int j = threadIdx.x + HIST_STAGED; j < len; j += NT) {
        const int t = __ldg(ids + j);
        if (t >= 0 && t < V) {
            const uint32_t bit = 1u << (t & 31);
            if (!(*(volatile uint32_t *)&hs.bitmap[t >> 5] & bit)) atomicOr(&hs.bitmap[t >> 5], bit);
        }
    }
    __syncthreads();
    // coarse exclusive prefix: one entry per 8 words; ncoarse <= 2048 for V <= 2^19
    uint32_t carry = 0;
    for (int base = 0; base < ncoarse; base += NT) {
        int cb = base + threadIdx.x;
        uint32_t pc = 0;
        if (cb < ncoarse) {
            if ((cb << 3) + 8 <= nwords) {
                const uint4 w0 = *(const uint4 *)&hs.bitmap[cb << 3], w1 = *(const uint4 *)&hs.bitmap[(cb << 3) + 4];
                pc = __popc(w0.x) + __popc(w0.y) + __popc(w0.z) + __popc(w0.w) + __popc(w1.x) + __popc(w1.y) + __popc(w1.z) + __popc(w1.w);
            } else {
                for (int w = cb << 3; w < nwords; ++w) pc += __popc(hs.bitmap[w]);
            }
        }
        uint32_t tot;
        uint32_t ex = block_exscan_u32(s, pc, tot);
        if (cb < ncoarse) hs.coarse[cb] = carry + ex;
        carry += tot;
    }
    const uint32_t U = carry;               // distinct valid ids
    uint32_t *cnt;
    bool ok = true;
    if (U <= CNT_CAP) cnt = hs.counts;
    else if (ws && ws_off >= 0 && ws_off + (int64_t)U <= ws_cap) cnt = ws + ws_off;
    else { cnt = nullptr; ok = false; }
    c.bitmap = hs.bitmap; c.coarse = hs.coarse; c.counts = cnt; c.n_distinct = U; c.ncoarse = ncoarse;
    if (!ok) return false;
    for (uint32_t u = threadIdx.x; u < U; u += NT) cnt[u] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < nst; j += NT) {
        const int t = staged[j];
        if (t >= 0 && t < V && j >= out_start) atomicAdd(&cnt[hist_rank(c, t)], 1u);
    }
    for (int j = threadIdx.x + HIST_STAGED; j < len; j += NT) {
        int t = __ldg(ids + j);
        if (t >= 0 && t < V && j >= out_start) atomicAdd(&cnt[hist_rank(c, t)], 1u);
    }
    __syncthreads();
    return true;
}

// token id of the r-th distinct history id (r < n_distinct), i.e. the r-th set bit of the bitmap
__device__ int hist_id_of_rank(const RowCtx &c, uint32_t r) {
    int lo = 0, hi = c.ncoarse - 1;            // last coarse block whose prefix is <= r
    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (c.coarse[mid] <= r) lo = mid; else hi = mid - 1; }
    uint32_t rem = r - c.coarse[lo];
    int w = lo << 3;
    for (;;) { const uint32_t pc = __popc(c.bitmap[w]); if (rem < pc) break; rem -= pc; ++w; }
    return (w << 5) + (int)__fns(c.bitmap[w], 0, (int)rem + 1);
}

// -ln E of token i for the general path's race, out of line with plain arguments only: the long
// Philox chain gets registers of its own and no structure of the caller is touched.
__device__ __noinline__ float race_nle(uint64_t seed, uint32_t R, uint64_t step, const float *exp1_row, int i) {
    if (exp1_row) return -logf(__ldg(exp1_row + i));
    return neg_log_exp1_fast(race_word(seed, R, step, i));
}

// ------------------------------------------------------------------ general path: histogram selection
//
// For rows the candidate path does not take (top-p without top-k, no cuts at all, a top-k above
// 256, or a candidate list that would overflow).  The kept set is a prefix of the total order, i.e.
// { t : C(t) >= C_cut }; the cut is found exactly with a few passes over the row (re-read from L2):
//   pass 0  the largest composite (z_max and its id) and the number of finite scores;
//   pass 1  a 2048-bin histogram (count, and 2^40 fixed-point mass) over value-linear bins of
//           z_max - z (1/32 wide), so that elements spread over many bins;
//   cut     the bin in which the wanted rank or mass falls; its elements are gathered into shared
//           memory and the exact position is found there (a bin too full for that is first narrowed
//           with composite-linear histograms over the row);
//   final   the race over the kept set, its mass and its size.

struct HistBins {
    uint32_t *cnt;   // HIST_BINS element counts
    uint32_t *limb;  // 3 x HIST_BINS: the bins' masses as three 14-bit limbs (32-bit shared-memory
                     // adds are native and a limb sum cannot overflow for fewer than 2^18 elements;
                     // a 64-bit add would be a compare-and-swap loop)
    u64 *list;       // GL_CAP composites gathered from the row
    u64 *acc;        // SEL_ACC bins for the on-chip search in the list
};
__device__ __forceinline__ void hist_add_mass(const HistBins &h, int q, u64 e) {
    const uint32_t l0 = (uint32_t)e & 0x3FFFu, l1 = (uint32_t)(e >> 14) & 0x3FFFu, l2 = (uint32_t)(e >> 28);
    if (l0) atomicAdd(&h.limb[q], l0);
    if (l1) atomicAdd(&h.limb[HIST_BINS + q], l1);
    if (l2) atomicAdd(&h.limb[2 * HIST_BINS + q], l2);
}
__device__ __forceinline__ u64 hist_mass(const HistBins &h, int q) {
    return (u64)h.limb[q] + ((u64)h.limb[HIST_BINS + q] << 14) + ((u64)h.limb[2 * HIST_BINS + q] << 28);
}
__device__ __forceinline__ void hist_clear(const HistBins &h) {
    for (int q = threadIdx.x; q < HIST_BINS; q += NT) { h.cnt[q] = 0; h.limb[q] = 0; h.limb[HIST_BINS + q] = 0; h.limb[2 * HIST_BINS + q] = 0; }
}

constexpr int GL_CAP = 2048;
constexpr float BIN_SCALE = 32.0f;      // bins per unit of z

struct RowParams {
    float T, top_p, min_p;
    int32_t top_k;
    uint64_t seed;
    uint32_t R;
    bool greedy;
    double ln_min_p;   // ln(min_p) in fp64, once per row (0 when min-p is off)
};

struct RowOut {
    int32_t token; float logprob; int32_t n_keep, n_topk; uint32_t status;
};

// smallest fp32 z with (double)z - (double)zmax >= ln(min_p), as an order key
__device__ uint32_t minp_key(float zmax, double thr) {
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

// Mass of an element at distance d = z - zmax <= 0 in 2^40 fixed point, from the hardware
// exponential (the general path runs it once per element and pass; its relative error of ~2^-21
// is far inside the logprob tolerance).  Used by every step of the general path alike.
__device__ __forceinline__ u64 mass_gen(float d) {
    return d < -28.5f ? 0ull : __float2ull_rn(__expf(d) * FX_SCALE);
}

// Mass of the whole row, sum of exp(z - zmax) over its finite scores in 2^40 fixed point: the
// normaliser of the log-probabilities in the full-vocabulary mode.  One more pass over the row (it
// was just read, so mostly from L2), four loads in flight; vectors with nothing within 29 of the
// maximum carry no mass and are skipped by the packed test of the candidate path; the masses of a
// vector are added in fp32 (a fixed order) and turned into fixed point once.  The same in every thread.
template <int DT>
__device__ u64 full_vocab_mass(BlockScratch &s, const RowCtx &c, float zmax) {
    typedef Elem<DT> E;
    typedef VecTest<DT> T;
    const int V = c.V;
    const uintptr_t addr = (uintptr_t)c.row;
    int head = (int)(((16u - (uint32_t)(addr & 15u)) & 15u) / E::SIZE);
    if (head > V) head = V;
    const int nvec = (V - head) / E::PER_VEC;
    const uint4 *vp = (const uint4 *)((const char *)c.row + (size_t)head * E::SIZE);
    const uint32_t thr = T::raw_threshold(key_of(zmax - 29.0f), c.invT);
    u64 local = 0;
    for (int v0 = threadIdx.x; v0 < nvec; v0 += 4 * NT) {
        uint4 q[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) q[u] = (v0 + u * NT < nvec) ? __ldg(vec_ptr<DT>(c, vp, v0 + u * NT)) : T::fill();
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int v = v0 + u * NT;
            if (v >= nvec) break;
            if (!T::may_pass(q[u], thr, c.invT)) continue;
            const int i0 = head + v * E::PER_VEC;
            uint32_t m = 0;
            if (c.has_hist) m = __funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31);
            float acc = 0.0f;
#pragma unroll
            for (int e = 0; e < E::PER_VEC; ++e) {
                const float d = __fsub_rn(__fmul_rn(E::get(q[u], e), c.invT), zmax);
                if (!((m >> e) & 1u) && d >= -28.5f) acc += __expf(d);
            }
            local += __float2ull_rn(acc * FX_SCALE);
        }
    }
    for_each_score_rest<DT>(c, head, nvec, [&](int, float z) {
        const float d = __fsub_rn(z, zmax);
        if (d > -3.0e38f) local += mass_gen(d);         // -inf (and NaN) carry no mass
    });
    return block_sum_u64(s, local);
}

// value-linear bin of a finite score z <= zmax; monotone: a larger z never gets a larger bin
__device__ __forceinline__ int bin_of(float z, float zmax) {
    int b = __float2int_rz(__fsub_rn(zmax, z) * BIN_SCALE);
    return b < 0 ? 0 : (b > HIST_BINS - 1 ? HIST_BINS - 1 : b);
}
__device__ __forceinline__ int bitlen64(u64 v) { return 64 - __clzll((long long)v); }

// Finds the first bin (from bin 0) at which the running total of the steering histogram reaches
// `target` (1 <= target <= grand total).  Gives the totals of both histograms strictly before it.
__device__ bool find_prefix_bin(BlockScratch &s, const HistBins &h, bool by_mass, bool have_mass, u64 target,
                                int &bin, u64 &cnt_before, u64 &mass_before) {
    constexpr int PER = HIST_BINS / NT;
    u64 lc = 0, lm = 0;
#pragma unroll
    for (int q = 0; q < PER; ++q) { lc += h.cnt[threadIdx.x * PER + q]; if (have_mass) lm += hist_mass(h, threadIdx.x * PER + q); }
    u64 totc, totm = 0;
    u64 runc = block_exscan_u64(s, lc, totc);
    u64 runm = have_mass ? block_exscan_u64(s, lm, totm) : 0ull;
    if (threadIdx.x == 0) s.found_digit = 0xFFFFFFFFu;
    __syncthreads();
    const u64 run = by_mass ? runm : runc, loc = by_mass ? lm : lc;
    if (run < target && target <= run + loc) {
        u64 rc = runc, rm = runm;
        for (int q = 0; q < PER; ++q) {
            const int bq = threadIdx.x * PER + q;
            const u64 vc = h.cnt[bq], vm = have_mass ? hist_mass(h, bq) : 0ull;
            const u64 r = by_mass ? rm : rc, v = by_mass ? vm : vc;
            if (r < target && target <= r + v) { s.found_digit = (uint32_t)bq; s.found_above = rc; s.bcast[2] = rm; break; }
            rc += vc; rm += vm;
        }
    }
    __syncthreads();
    if (s.found_digit == 0xFFFFFFFFu) return false;
    bin = (int)s.found_digit; cnt_before = s.found_above; mass_before = s.bcast[2];
    return true;
}

// Gathers the composites accepted by `take` into h.list (at most GL_CAP are stored); returns how many
// were accepted, and their smallest and largest composite.
template <int DT, class F>
__device__ int gather_if(BlockScratch &s, const HistBins &h, const RowCtx &c, F &&take, u64 &cmin, u64 &cmax) {
    if (threadIdx.x == 0) s.list_cnt = 0;
    __syncthreads();
    u64 mn = ~0ull, mx = 0;
    for_each_score<DT>(c, [&](int i, float z) {
        const u64 C = comp_of(key_of(z), i);
        if (take(C, z)) {
            const uint32_t slot = atomicAdd(&s.list_cnt, 1u);
            if (slot < (uint32_t)GL_CAP) h.list[slot] = C;
            mn = C < mn ? C : mn; mx = C > mx ? C : mx;
        }
    });
    cmax = block_max_u64(s, mx);
    cmin = ~block_max_u64(s, ~mn);
    return (int)s.list_cnt;
}

// On-chip: in h.list[0..n) (distinct composites, n <= GL_CAP) find the composite at which the running
// total, taken from the largest composite down over those within [lo, hi], first reaches `target` --
// counting elements (by_mass = false) or their masses.  The list is sorted in place (a bitonic network
// over the next power of two, every thread a few compare-exchanges per step) and the totals are a
// prefix sum over the sorted order: the cost does not depend on how the composites are spread, and
// equal keys, which quantised logits produce in their hundreds, cost nothing extra.
// (out of line, and given plain pointers only, so that it neither shapes the register allocation of
// its callers nor forces their structures into local memory)
__device__ __noinline__ u64 list_resolve(BlockScratch *sp, u64 *list, int n, bool by_mass, u64 target, u64 lo, u64 hi, float zmax) {
    BlockScratch &s = *sp;
    struct { u64 *list; } h = {list};
    int P = 2;
    while (P < n) P <<= 1;
    for (int i = threadIdx.x; i < P; i += NT) {
        const u64 C = i < n ? h.list[i] : 0ull;
        h.list[i] = (C >= lo && C <= hi) ? C : 0ull;            // 0 sorts last and counts for nothing
    }
    __syncthreads();
    for (int k = 2; k <= P; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int t = threadIdx.x; t < (P >> 1); t += NT) {
                const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1)), l = i | j;
                const u64 a = h.list[i], b2 = h.list[l];
                const bool desc = (i & k) == 0;                  // final order: descending
                if (desc ? a < b2 : a > b2) { h.list[i] = b2; h.list[l] = a; }
            }
            __syncthreads();
        }
    }
    // each thread owns a run of consecutive sorted entries
    const int per = (P + NT - 1) / NT;
    const int q0 = threadIdx.x * per, q1 = min(P, q0 + per);
    u64 local = 0;
    for (int q = q0; q < q1; ++q) {
        const u64 C = h.list[q];
        if (C) local += by_mass ? mass_gen(__fsub_rn(unkey((uint32_t)(C >> 32)), zmax)) : 1ull;
    }
    u64 tot;
    u64 run = block_exscan_u64(s, local, tot);
    if (threadIdx.x == 0) { s.bcast[3] = lo; }                   // target beyond the list: keep all of it
    __syncthreads();
    if (run < target && target <= run + local) {
        for (int q = q0; q < q1; ++q) {
            const u64 C = h.list[q];
            if (!C) break;
            run += by_mass ? mass_gen(__fsub_rn(unkey((uint32_t)(C >> 32)), zmax)) : 1ull;
            if (run >= target) { s.bcast[3] = C; break; }
        }
    }
    __syncthreads();
    const u64 res = s.bcast[3];
    __syncthreads();
    return res;
}

// Exact cut inside the row: the composite at which the running total (count or mass, from the top of
// the order, over elements with C >= floorC) first reaches `target`, given that it falls in value bin
// `bin` and that `before` of the total lies in the bins ahead of it.
template <int DT>
__device__ u64 resolve_cut(BlockScratch &s, const HistBins &h, const RowCtx &c, float zmax, int bin, bool by_mass,
                           u64 target, u64 before, u64 floorC, bool &hist_clobbered) {
    u64 rel = target - before;
    u64 lo, hi;
    int n = gather_if<DT>(s, h, c, [&](u64 C, float z) { return C >= floorC && (C >> 32) < KEY_POS_INF && bin_of(z, zmax) == bin; }, lo, hi);
    // a bin too full for the list is narrowed with composite-linear histograms over the row
    for (int it = 0; it < 8 && n > GL_CAP; ++it) {
        const u64 width = hi - lo;
        const int shift = width < (u64)HIST_BINS ? 0 : bitlen64(width) - 11;
        hist_clobbered = true;                               // the value histograms are overwritten
        hist_clear(h);
        __syncthreads();
        for_each_score<DT>(c, [&](int i, float z) {
            const u64 C = comp_of(key_of(z), i);
            if (C >= lo && C <= hi && C >= floorC) {
                const uint32_t q = (uint32_t)((hi - C) >> shift);
                atomicAdd(&h.cnt[q], 1u);
                if (by_mass) hist_add_mass(h, (int)q, mass_gen(__fsub_rn(z, zmax)));
            }
        });
        __syncthreads();
        int sub; u64 cb, mb;
        if (!find_prefix_bin(s, h, by_mass, by_mass, rel, sub, cb, mb)) return lo > floorC ? lo : floorC;
        rel -= by_mass ? mb : cb;
        const u64 nhi = hi - ((u64)sub << shift);
        if (shift == 0) return nhi;
        const u64 span = (1ull << shift) - 1ull;
        const u64 nlo = (nhi - lo > span) ? nhi - span : lo;
        n = (int)h.cnt[sub];
        __syncthreads();
        lo = nlo; hi = nhi;
        if (n <= GL_CAP) {
            u64 l2, h2;
            n = gather_if<DT>(s, h, c, [&](u64 C, float) { return C >= lo && C <= hi && C >= floorC; }, l2, h2);
            lo = l2; hi = h2;
        }
    }
    if (n > GL_CAP) return lo > floorC ? lo : floorC;        // not reachable: composites are distinct
    if (n < 1) return floorC;
    return list_resolve(&s, h.list, n, by_mass, rel, lo, hi, zmax);
}

template <int DT, class A>
__device__ __forceinline__ void general_path(BlockScratch &s, const HistBins &h, const RowCtx &c, const RowParams &rp,
                                             const A &a, int b, RowOut &out) {
    const int V = c.V;
    // pass 0: the largest key and the number of finite scores
    uint32_t kbest = 0, nfin_local = 0;
    pass0_max_count<DT>(c, kbest, nfin_local);
    const uint32_t kmax = (uint32_t)block_max_u64(s, kbest);
    const u64 n_fin = block_sum_u64(s, nfin_local);
    const float zmax = unkey(kmax);
    out.status |= ALBIREO_ROW_GENERAL_PATH;
    // the first element of the order: the lowest id among the largest keys (one more pass, only when asked for)
    auto top_id = [&]() -> int {
        uint32_t best = 0;
        for_each_score<DT>(c, [&](int i, float z) { if (key_of(z) == kmax) { const uint32_t v = ~(uint32_t)i; best = v > best ? v : best; } });
        return (int)~(uint32_t)block_max_u64(s, best);
    };

    const bool full_lp = (a.flags & ALBIREO_FLAG_LOGPROB_FULL_VOCAB) != 0;
    if (threadIdx.x == 0) s.nfin_cap = (uint32_t)(n_fin < (u64)ALBIREO_MAX_NUM_TOP + 1 ? n_fin : (u64)ALBIREO_MAX_NUM_TOP + 1);
    const u64 Cfin = (u64)KEY_MIN_FINITE << 32;
    const int top_k = rp.greedy ? 1 : rp.top_k;          // (a greedy row gets here only for the whole-vocabulary list)
    const bool want_k = top_k >= 1 && top_k < V && (u64)top_k < n_fin;
    const bool want_minp = !rp.greedy && rp.min_p > 0.0f;
    const bool want_topp = !rp.greedy && rp.top_p < 1.0f;
    const bool want_top_list = a.num_top > 0;
    bool have_hist = false, have_mass = false;           // which value histograms are current
    auto build_hist = [&](bool with_cnt, bool with_mass) {
        hist_clear(h);
        __syncthreads();
        for_each_score<DT>(c, [&](int, float z) {
            const float d = __fsub_rn(zmax, z);               // >= 0 for finite z; inf / NaN otherwise
            if (d < 3.0e38f) {
                int q = __float2int_rz(d * BIN_SCALE);
                q = q > HIST_BINS - 1 ? HIST_BINS - 1 : q;
                if (with_cnt) atomicAdd(&h.cnt[q], 1u);
                if (with_mass) { const u64 e = mass_gen(-d); if (e) hist_add_mass(h, q, e); }
            }
        });
        __syncthreads();
        have_hist = with_cnt; have_mass = with_mass;
    };
    // The top-N list: the first min(num_top, members) entries, in order, of the set { C >= floorC } (the
    // final kept set of `members` elements; in the full-vocabulary mode every finite score of the row).
    auto write_top_list = [&](u64 members, u64 floorC, double lnS) {
        const u64 want = members < (u64)a.num_top ? members : (u64)a.num_top;
        u64 CN = floorC;
        if (want < members) {
            if (!have_hist) build_hist(true, false);
            int bin; u64 cb, mb;
            bool clobbered = false;
            if (find_prefix_bin(s, h, false, false, want, bin, cb, mb))
                CN = resolve_cut<DT>(s, h, c, zmax, bin, false, want, cb, floorC, clobbered);
            if (clobbered) have_hist = have_mass = false;
        }
        u64 lo, hi;
        const int n = gather_if<DT>(s, h, c, [&](u64 C, float) { return C >= CN && (C >> 32) < KEY_POS_INF; }, lo, hi);
        const int m = n < ALBIREO_MAX_NUM_TOP ? n : ALBIREO_MAX_NUM_TOP;
        if ((int)threadIdx.x < m) {
            const u64 C = h.list[threadIdx.x];
            int rank = 0;
            for (int q = 0; q < m; ++q) rank += h.list[q] > C;
            if (rank < a.num_top) {
                const int64_t o = (int64_t)b * a.num_top + rank;
                a.out_top_ids[o] = comp_idx(C);
                a.out_top_logprobs[o] = (members == 1 && !full_lp) ? 0.0f : (float)(((double)unkey((uint32_t)(C >> 32)) - (double)zmax) - lnS);
            }
        }
        __syncthreads();
    };
    // Greedy rows (and rows with a single finite score) need the arg max only -- unless the list over
    // the whole vocabulary is wanted: then they go through the cuts below as top_k = 1.
    if ((rp.greedy || n_fin <= 1) && !(full_lp && want_top_list)) {
        out.token = top_id(); out.logprob = 0.0f; out.n_keep = 1; out.n_topk = 1;
        if (full_lp) out.logprob = (float)-(log((double)full_vocab_mass<DT>(s, c, zmax)) - LN2_40);
        if (a.dbg_topk_ids && a.dbg_cap >= 1 && threadIdx.x == 0) a.dbg_topk_ids[(int64_t)b * a.dbg_cap] = out.token;
        if (want_top_list && threadIdx.x == 0) {
            a.out_top_ids[(int64_t)b * a.num_top] = out.token;
            a.out_top_logprobs[(int64_t)b * a.num_top] = out.logprob;
        }
        return;
    }
    if (want_k || want_topp) build_hist(want_k, want_topp);

    // top-k stage
    u64 C1 = Cfin;
    u64 n_topk = n_fin;
    if (want_k) {
        n_topk = (u64)top_k;
        int bin; u64 cb, mb;
        const bool find_ok = find_prefix_bin(s, h, false, want_topp, n_topk, bin, cb, mb);
        bool clobbered = false;
        if (find_ok) C1 = resolve_cut<DT>(s, h, c, zmax, bin, false, n_topk, cb, Cfin, clobbered);
        if (clobbered) have_hist = have_mass = false;
        if ((a.flags & ALBIREO_FLAG_TOPK_KEEP_TIES) && !rp.greedy) {
            // every id of the k-th largest key stays; how many that makes takes a count over the row
            C1 &= 0xFFFFFFFF00000000ull;
            const uint32_t k1 = (uint32_t)(C1 >> 32);
            uint32_t local = 0;
            for_each_score<DT>(c, [&](int, float z) { const uint32_t kk = key_of(z); local += (kk >= k1 && kk < KEY_POS_INF); });
            n_topk = block_sum_u64(s, local);
        }
        if (want_topp && !have_mass) build_hist(false, true);
    }
    out.n_topk = (int32_t)n_topk;
    if (a.dbg_topk_ids && top_k >= 1 && top_k < V && n_topk <= (u64)a.dbg_cap) {
        if (threadIdx.x == 0) s.list_cnt = 0;
        __syncthreads();
        int32_t *dst = a.dbg_topk_ids + (int64_t)b * a.dbg_cap;
        for_each_score<DT>(c, [&](int i, float z) {
            if (comp_of(key_of(z), i) >= C1) { uint32_t slot = atomicAdd(&s.list_cnt, 1u); if (slot < (uint32_t)a.dbg_cap) dst[slot] = i; }
        });
        __syncthreads();
    }
    // min-p: a value threshold, never above the top element
    if (want_minp) {
        u64 Cm = (u64)minp_key(zmax, rp.ln_min_p) << 32;
        if ((uint32_t)(Cm >> 32) > kmax) Cm = comp_of(kmax, top_id());     // floor above the maximum: the first element alone
        if (Cm > C1) C1 = Cm;
    }
    // top-p on the mass of the survivors
    u64 C2 = C1;
    if (want_topp) {
        u64 Sp = 0;
        if (C1 == Cfin) {
            u64 lm = 0;
            for (int q = threadIdx.x; q < HIST_BINS; q += NT) lm += hist_mass(h, q);
            Sp = block_sum_u64(s, lm);
        } else {
            u64 lm = 0;
            const uint32_t k1 = (uint32_t)(C1 >> 32); const int id1 = comp_idx(C1);
            for_each_score<DT>(c, [&](int i, float z) { const uint32_t k = key_of(z); if (k > k1 || (k == k1 && (uint32_t)i <= (uint32_t)id1)) lm += mass_gen(__fsub_rn(z, zmax)); });
            Sp = block_sum_u64(s, lm);
        }
        double t = ceil((double)rp.top_p * (double)Sp);
        u64 target = t <= 1.0 ? 1ull : (u64)t;
        if (target > Sp) target = Sp;
        if (target < 1) target = 1;
        int bin; u64 cb, mb;
        bool clobbered = false;
        if (find_prefix_bin(s, h, true, true, target, bin, cb, mb))
            C2 = resolve_cut<DT>(s, h, c, zmax, bin, true, target, mb, C1, clobbered);
        if (C2 < C1) C2 = C1;
        if (clobbered) have_hist = have_mass = false;
    }

    // final pass: mass of the kept set, its size, and the race.  An element whose score cannot
    // beat the thread's best even with the luckiest draw (-ln E <= 23 for the generator's words) is skipped.
    // The race term is a long computation that only kept elements need, and in a wide kept set they
    // are scattered over the lanes of a warp: running it in place would execute it for almost every
    // element position with few lanes active.  So each thread queues its contenders in shared memory
    // (a private queue, over the histograms, which are done with) and the warp works the queues off
    // together whenever one of them runs full: then most lanes have an entry to work on.
    u64 S_local = 0, g_best = 0;
    uint32_t n_local = 0;
    float best_g = -3.0e38f;
    const uint32_t k2 = (uint32_t)(C2 >> 32);
    const int id2 = comp_idx(C2);
    const float *exp1_row = a.exp1 ? a.exp1 + (int64_t)b * a.exp1_stride : nullptr;
    const float luck = exp1_row ? 104.0f : 23.0f;        // largest -ln E: a table may hold any positive fp32
    have_hist = have_mass = false;
    __syncthreads();
    constexpr int RQ_DEPTH = 12;                         // 8 elements of a vector on top of at most 4 left over
    u64 *rq = (u64 *)h.cnt + threadIdx.x;                // entry j of this thread at rq[j * NT]: 48 KiB in all
    int qn = 0;
    auto race_one = [&](int i, float d) {
        if (d + luck >= best_g) {
            const float g = d + race_nle(rp.seed, rp.R, a.step, exp1_row, i);
            const u64 G = ((u64)orderable_f32(g) << 32) | (uint32_t)(~(uint32_t)i);
            if (G > g_best) { g_best = G; best_g = g; }
        }
    };
    auto see = [&](int i, float z, bool may_queue) {
        const uint32_t k = key_of(z);
        if (k > k2 || (k == k2 && (uint32_t)i <= (uint32_t)id2)) {
            const float d = __fsub_rn(z, zmax);
            S_local += mass_gen(d);
            n_local += 1;
            if (d + luck >= best_g) {
                if (may_queue && qn < RQ_DEPTH) { rq[qn * NT] = ((u64)__float_as_uint(d) << 32) | (uint32_t)i; ++qn; }
                else race_one(i, d);
            }
        }
    };
    // called by whole warps: works the queues down until none holds more than `leave`
    auto drain = [&](int leave) {
        while (__any_sync(0xFFFFFFFFu, qn > leave)) {
            if (qn > 0) { --qn; const u64 e = rq[qn * NT]; race_one((int)(uint32_t)e, __uint_as_float((uint32_t)(e >> 32))); }
        }
    };
    {
        typedef Elem<DT> E;
        const uintptr_t addr = (uintptr_t)c.row;
        int head = (int)(((16u - (uint32_t)(addr & 15u)) & 15u) / E::SIZE);
        if (head > V) head = V;
        const int nvec = (V - head) / E::PER_VEC;
        const uint4 *vp = (const uint4 *)((const char *)c.row + (size_t)head * E::SIZE);
        for (int base = 0; base < nvec; base += 2 * NT) {            // the same trip count in every thread
            const int v0 = base + (int)threadIdx.x, v1 = v0 + NT;
            const uint4 q0 = v0 < nvec ? __ldg(vec_ptr<DT>(c, vp, v0)) : make_uint4(0, 0, 0, 0);
            const uint4 q1 = v1 < nvec ? __ldg(vec_ptr<DT>(c, vp, v1)) : q0;
#pragma unroll 1
            for (int u = 0; u < 2; ++u) {
                const int v = u ? v1 : v0;
                if (v < nvec) {
                    const uint4 &q = u ? q1 : q0;
                    const int i0 = head + v * E::PER_VEC;
                    uint32_t m = 0;
                    if (c.has_hist) m = __funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31);
#pragma unroll
                    for (int e = 0; e < E::PER_VEC; ++e)
                        if (!((m >> e) & 1u)) see(i0 + e, __fmul_rn(E::get(q, e), c.invT), true);
                }
                drain(RQ_DEPTH - E::PER_VEC);
            }
        }
        for_each_score_rest<DT>(c, head, nvec, [&](int i, float z) { see(i, z, true); });
        drain(0);
    }
    const u64 S_fx = block_sum_u64(s, S_local);
    const u64 n_keep = block_sum_u64(s, n_local);
    const u64 G = block_max_u64(s, g_best);
    const int tok = comp_idx(G);
    const double lnS = log((double)(full_lp ? full_vocab_mass<DT>(s, c, zmax) : S_fx)) - LN2_40;
    float z_tok = score_of(c, tok, Elem<DT>::load(elem_ptr<DT>(c, tok), 0));
    out.token = tok;                                   // (a single kept element wins its own race)
    out.logprob = (n_keep == 1 && !full_lp) ? 0.0f : (float)(((double)z_tok - (double)zmax) - lnS);
    out.n_keep = (int32_t)n_keep;

    if (want_top_list) write_top_list(full_lp ? (u64)s.nfin_cap : n_keep, full_lp ? ((u64)KEY_MIN_FINITE << 32) : C2, lnS);
}

// The general path as a function of its own: its registers are allocated apart from the streaming
// path's (the whole kernel is held to 64 per thread) and its size does not shape that path's code.
// The row's context travels by value, the few launch arguments it needs through shared memory
// (BlockScratch::ga, written by the caller before the barrier in front of the call).
template <int DT>
__device__ __noinline__ RowOut general_path_call(BlockScratch *sp, unsigned char *smem, RowCtx c, RowParams rp, int b, uint32_t status) {
    HistBins h;
    h.cnt = (uint32_t *)smem;
    h.limb = (uint32_t *)(smem + HIST_BINS * 4);
    h.list = (u64 *)(smem + HIST_BINS * 16);
    h.acc = h.list + GL_CAP;
    RowOut out;
    out.token = 0; out.logprob = 0.0f; out.n_keep = 0; out.n_topk = 0; out.status = status;
    general_path<DT>(*sp, h, c, rp, sp->ga, b, out);
    return out;
}

// ------------------------------------------------------------------ TMA bulk-copy ring
//
// The row is streamed through a ring of shared-memory stages filled by 1-D bulk async
// copies (cp.async.bulk, completion on an mbarrier), several tiles ahead of the scan.
// Every wait is bounded: on expiry the row reports ALBIREO_ROW_TIMEOUT and the CTA drains
// its copies and leaves.

struct Ring {
    // source of the copies: vectors per piece of the row and the distance between pieces (a row in
    // one piece: vps covers the whole row)
    int vps;
    const char *const *seg_base;
    unsigned char *buf;     // nstages * STAGE_BYTES, 128-byte aligned
    uint64_t *bar;          // one mbarrier per stage
    int nstages;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, int cap = WAIT_CAP) {
    for (int it = 0; it < cap; ++it) if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// global -> shared bulk copy; src and dst 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_g2s(void *dst, const void *src, uint32_t bytes, uint64_t *bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// copies vectors [v0, v0 + nv) of the row to dst, piece by piece; the bytes were announced to `bar`
__device__ __forceinline__ void ring_copy(const Ring &rg, void *dst, const uint4 *vp, int v0, int nv, uint64_t *bar) {
    if (rg.vps == 0x7FFFFFFF) { bulk_g2s(dst, vp + v0, (uint32_t)nv * 16u, bar); return; }    // one piece
    unsigned char *d = (unsigned char *)dst;
    int j = v0 / rg.vps, off = v0 - j * rg.vps;
    while (nv > 0) {
        const int n1 = nv < rg.vps - off ? nv : rg.vps - off;
        bulk_g2s(d, (const uint4 *)rg.seg_base[j] + off, (uint32_t)n1 * 16u, bar);
        d += (size_t)n1 * 16; nv -= n1; ++j; off = 0;
    }
}
// issues the copy of tile t (called by one thread)
__device__ __forceinline__ void ring_issue(const Ring &rg, const uint4 *vp, int nvec, int t, int st) {
    const int v0 = t * (NT * TILE_VECS);
    int nv = nvec - v0; if (nv > NT * TILE_VECS) nv = NT * TILE_VECS;
    mbar_expect_tx(&rg.bar[st], (uint32_t)nv * 16u);
    ring_copy(rg, rg.buf + (size_t)st * STAGE_BYTES, vp, v0, nv, &rg.bar[st]);
}
// Tile 0 arrives in two copies: its first NT vectors (the warm-up slice, one vector per thread) on
// their own mbarrier so that the threshold can be set up while the rest is still in flight.
__device__ __forceinline__ void ring_issue_first(const Ring &rg, const uint4 *vp, int nvec) {
    const int na = nvec < NT ? nvec : NT;
    int nb = nvec - na; if (nb > NT * (TILE_VECS - 1)) nb = NT * (TILE_VECS - 1);
    mbar_expect_tx(&rg.bar[MAX_STAGES - 1], (uint32_t)na * 16u);
    ring_copy(rg, rg.buf, vp, 0, na, &rg.bar[MAX_STAGES - 1]);
    if (nb > 0) {
        mbar_expect_tx(&rg.bar[0], (uint32_t)nb * 16u);
        ring_copy(rg, rg.buf + (size_t)na * 16, vp, na, nb, &rg.bar[0]);
    } else {
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&rg.bar[0])) : "memory");
    }
}
// waits for the copies of tiles [t0, t1) so that the CTA may leave or reuse the ring
__device__ void ring_drain(const Ring &rg, int t0, int t1) {
    for (int t = t0; t < t1; ++t) mbar_wait(&rg.bar[t % rg.nstages], (uint32_t)(t / rg.nstages) & 1u);
}

// ------------------------------------------------------------------ candidate path
//
// One streaming pass over the row.  A conservative threshold tau (an order key) is kept
// such that every element of the final kept set has key >= tau: (a lower bound of) the
// k-th largest key seen so far (top-k), and/or the min-p floor below the running maximum.
// Elements below tau are dropped by a cheap vector test; the rest are checked exactly and
// appended to a small on-chip candidate list, which is finally sorted and cut.
// Penalised tokens never enter through the stream (their raw value is not their score):
// they are evaluated from the history bitmap after the stream.

struct CandSmem {
    u64 *cand;        // CAND_CAP composites
    uint32_t *hist;   // SEL_BINS bins while selecting
    // scratch of the final stage, in the (by then idle) ring: sorted composites, masses, race scores
    u64 *sorted, *efx, *gsc;
};

constexpr int SEL_BINS = NT;            // one bin per thread

__device__ __forceinline__ uint32_t warp_incl_scan_u32(uint32_t v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { uint32_t t = __shfl_up_sync(0xFFFFFFFFu, v, o); if (lane >= o) v += t; }
    return v;
}

// One histogram pass over cand[0..n) restricted to keys in [lo, hi]: finds the bin that
// holds the k-th largest such key.  Returns false if fewer than k keys are in range.
// On success [lo, hi] is narrowed to that bin and k to the rank inside it; `shift` tells
// the bin width (0: the bin is a single key, i.e. lo is exactly the k-th largest key).
__device__ bool cand_select_pass(BlockScratch &s, const CandSmem &cs, int n, uint32_t &k, uint32_t &lo, uint32_t &hi, int &shift,
                                 bool zeroed = false) {
    const uint32_t width = hi - lo;
    shift = width < (uint32_t)SEL_BINS ? 0 : (32 - __clz(width)) - 9;
    if (!zeroed) {          // (a caller that zeroed the bins and found_digit before its last barrier skips this)
        cs.hist[threadIdx.x] = 0;
        if (threadIdx.x == 0) s.found_digit = 0xFFFFFFFFu;
        __syncthreads();
    }
    for (int i = threadIdx.x; i < n; i += NT) {
        uint32_t key = (uint32_t)(cs.cand[i] >> 32);
        if (key >= lo && key <= hi) atomicAdd(&cs.hist[(key - lo) >> shift], 1u);
    }
    __syncthreads();
    // thread t owns bin SEL_BINS-1-t, so thread order is descending key order
    const uint32_t mine = cs.hist[SEL_BINS - 1 - threadIdx.x];
    const uint32_t inc = warp_incl_scan_u32(mine);
    if ((threadIdx.x & 31) == 31) s.r32a[threadIdx.x >> 5] = inc;
    __syncthreads();
    uint32_t base = 0;
    const int wid = threadIdx.x >> 5;
#pragma unroll
    for (int w = 0; w < NWARPS; ++w) base += (w < wid) ? s.r32a[w] : 0u;
    const uint32_t above = base + inc - mine;
    if (above < k && k <= above + mine) { s.found_digit = SEL_BINS - 1 - threadIdx.x; s.found_cnt = above; }
    __syncthreads();
    const uint32_t digit = s.found_digit;
    const uint32_t fcnt = s.found_cnt;
    // (everybody has the result before the next pass, or anybody else, resets it: a thread that read
    // the reset value instead would leave the caller's loop early and miss that pass's barriers)
    __syncthreads();
    if (digit == 0xFFFFFFFFu) return false;
    k -= fcnt;
    const uint32_t nlo = lo + (digit << shift);
    uint32_t nhi = nlo + ((1u << shift) - 1u);
    if (nhi > hi || nhi < nlo) nhi = hi;
    lo = nlo; hi = nhi;
    return true;
}

// Lower bound t of the k-th largest key in [lo, hi]: count(key >= t) >= k.  One pass when the
// keys spread over the bins; an outlier that stretches the range leaves most keys in one bin, and
// then up to two more passes narrow that bin.
__device__ uint32_t cand_select_approx(BlockScratch &s, const CandSmem &cs, int n, int k, uint32_t lo, uint32_t hi, bool zeroed = false) {
    uint32_t kk = (uint32_t)k; int shift = 1;
    for (int pass = 0; pass < 3 && shift != 0; ++pass) {
        if (!cand_select_pass(s, cs, n, kk, lo, hi, shift, zeroed && pass == 0)) break;   // on failure lo is unchanged
        const uint32_t pop = cs.hist[s.found_digit];
        __syncthreads();
        if (pop <= (uint32_t)(k / 4 + 8)) break;
    }
    return lo;
}
// The k-th largest key in [lo, hi] exactly (as many passes as the key range needs).
__device__ uint32_t cand_select_exact(BlockScratch &s, const CandSmem &cs, int n, int k, uint32_t lo, uint32_t hi) {
    uint32_t kk = (uint32_t)k; int shift = 1;
    for (int pass = 0; pass < 5 && shift != 0; ++pass)
        if (!cand_select_pass(s, cs, n, kk, lo, hi, shift)) break;
    return lo;
}

// keeps the candidates with key >= tkey (and drops empty slots); returns the new count
__device__ int cand_compact(BlockScratch &s, const CandSmem &cs, int n, uint32_t tkey) {
    constexpr int PER = CAND_CAP / NT;
    u64 mine[PER];
    uint32_t cnt = 0;
#pragma unroll
    for (int q = 0; q < PER; ++q) {
        int i = threadIdx.x + q * NT;
        mine[q] = (i < n) ? cs.cand[i] : 0ull;
        if ((uint32_t)(mine[q] >> 32) < tkey) mine[q] = 0ull;
        cnt += mine[q] != 0ull;
    }
    const uint32_t inc = warp_incl_scan_u32(cnt);
    __syncthreads();
    if (threadIdx.x == 0) s.cand_cnt = 0;
    __syncthreads();
    uint32_t base = 0;
    if ((threadIdx.x & 31) == 31 && inc) base = atomicAdd(&s.cand_cnt, inc);
    base = __shfl_sync(0xFFFFFFFFu, base, 31) + inc - cnt;
#pragma unroll
    for (int q = 0; q < PER; ++q) if (mine[q] != 0ull) cs.cand[base++] = mine[q];
    __syncthreads();
    return (int)s.cand_cnt;
}

// bit e set: element e of the vector is unpenalised and its score has key >= tau
template <int DT>
__device__ __forceinline__ uint32_t exact_pass_bits(const RowCtx &c, const uint4 &q, int i0, uint32_t tau_key) {
    typedef Elem<DT> E;
    uint32_t m = 0, bits = 0;
    if (c.has_hist) m = __funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31);
#pragma unroll
    for (int e = 0; e < E::PER_VEC; ++e) {
        uint32_t key = key_of(__fmul_rn(E::get(q, e), c.invT));
        if (key >= tau_key && !((m >> e) & 1u)) bits |= 1u << e;
    }
    return bits;
}

// key of the largest unpenalised score in a vector (0 if none), for the warm-up bound
template <int DT>
__device__ __noinline__ uint32_t masked_vmax_key(const RowCtx &c, uint4 q, int i0) {
    typedef Elem<DT> E;
    const uint32_t m = __funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31);
    uint32_t best = 0;
#pragma unroll
    for (int e = 0; e < E::PER_VEC; ++e) {
        if (m & (1u << e)) continue;
        uint32_t key = key_of(__fmul_rn(E::get(q, e), c.invT));
        best = key > best ? key : best;
    }
    return best;
}

// Single appends outside the streaming loop (scalar head/tail, penalised tokens).
__device__ __forceinline__ void cand_append_one(BlockScratch &s, const CandSmem &cs, u64 C) {
    cg::coalesced_group g = cg::coalesced_threads();
    uint32_t base = 0;
    if (g.thread_rank() == 0) base = atomicAdd(&s.cand_cnt, g.size());
    base = g.shfl(base, 0);
    const uint32_t slot = base + g.thread_rank();
    if (slot < (uint32_t)CAND_CAP) cs.cand[slot] = C; else s.overflow = 1u;
    atomicMax(&s.runmax, (uint32_t)(C >> 32));
}

// Final stage over the candidate list cand[0..n) (all distinct, n <= SORT_MAX), whose largest
// score is zmax.  Step 1 (all threads): each candidate's rank by counting (several threads share
// the comparisons of one candidate when n is small), its mass and its race score, written to its
// sorted position.  Step 2 (warp 0): the cuts as prefix operations and the argmax of the race.
// `full_fx` != 0: the log-probabilities are relative to that mass (the whole row's) instead of the kept set's.
__device__ void final_stage(BlockScratch &s, const CandSmem &cs, int n, int L6, float zmax, bool has_minp,
                            const RowParams &rp, const SampleArgs &a, int b, RowOut &out, u64 full_fx) {
    const int lane = threadIdx.x & 31;
    // `parts` threads share one candidate's comparisons; the threads after them (from the next warp
    // boundary on) take one candidate each for the race term and the mass, so those long dependent
    // chains run with full lanes and beside the rank loops instead of after them.
    int parts = 1;
    while (parts < 8 && ((n * parts * 2 + 31) & ~31) + n <= NT) parts *= 2;
    const int dstart = (n * parts + 31) & ~31;
    const bool dense_ok = dstart + n <= NT;
    const int j = threadIdx.x / parts, part = threadIdx.x % parts;
    float *nle = (float *)(cs.gsc + SORT_MAX);           // n race terms, then n masses (as u64) behind them
    u64 *mass = (u64 *)(nle + SORT_MAX);
    u64 C = 0;
    int rank = 0;
    if (j < n) {
        C = cs.cand[j];
#pragma unroll 4
        for (int q = part; q < n; q += parts) rank += cs.cand[q] > C;
    }
    {
        const int t = dense_ok ? (int)threadIdx.x - dstart : (part == 0 ? j : -1);
        if (t >= 0 && t < n) {
            const u64 Ct = cs.cand[t];
            nle[t] = a.exp1 ? -logf(__ldg(a.exp1 + (int64_t)b * a.exp1_stride + comp_idx(Ct)))
                            : neg_log_exp1_fast(race_word(rp.seed, rp.R, a.step, comp_idx(Ct)));
            mass[t] = mass_gen(__fsub_rn(unkey((uint32_t)(Ct >> 32)), zmax));
        }
    }
    for (int o = 1; o < parts; o <<= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, o);
    __syncthreads();
    bool in7 = false;
    if (j < n && part == 0) {
        const float z = unkey((uint32_t)(C >> 32));
        const float d = __fsub_rn(z, zmax);
        cs.sorted[rank] = C;
        cs.efx[rank] = mass[j];
        cs.gsc[rank] = ((u64)orderable_f32(d + nle[j]) << 32) | (uint32_t)C;
        in7 = rank < L6 && (!has_minp || ((double)z - (double)zmax >= rp.ln_min_p));
    }
    // min-p keeps a prefix of the order, at least one element (the barrier also publishes step 1)
    int L7 = __syncthreads_count(in7);
    if (L7 < 1) L7 = 1;
    if (a.dbg_topk_ids && L6 <= a.dbg_cap && (int)threadIdx.x < L6 && (rp.greedy || (rp.top_k >= 1 && rp.top_k < a.V)))
        a.dbg_topk_ids[(int64_t)b * a.dbg_cap + threadIdx.x] = comp_idx(cs.sorted[threadIdx.x]);
    if (threadIdx.x >= 32) return;

    const u64 *sorted = cs.sorted, *gsc = cs.gsc, *efx = cs.efx;
    int L8 = L7;
    int tok;
    float lp_tok, lnS;
    if (L7 <= 64) {
        // The usual case (a kept prefix of at most 64): lane l owns elements 2l and 2l + 1 and fetches
        // everything it will need of them in one round of shared-memory loads; the cut and the race are
        // then register work, ballots and shuffles only.  Same arithmetic as the general form below.
        const int qa = 2 * lane, qb = qa + 1;
        const bool va = qa < L7, vb = qb < L7;
        const u64 ea = va ? efx[qa] : 0ull, eb = vb ? efx[qb] : 0ull;
        const u64 ga = va ? gsc[qa] : 0ull, gb = vb ? gsc[qb] : 0ull;
        const u64 sa = va ? sorted[qa] : 0ull, sb = vb ? sorted[qb] : 0ull;
        const u64 s0 = __shfl_sync(0xFFFFFFFFu, sa, 0);
        const u64 local = ea + eb;
        u64 incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { u64 t2 = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += t2; }
        const u64 tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
        u64 S_fx = tot;
        if (!rp.greedy && rp.top_p < 1.0f) {
            double t = ceil((double)rp.top_p * (double)tot);
            u64 target = t <= 1.0 ? 1ull : (u64)t;
            if (target > tot) target = tot;
            // smallest prefix whose mass reaches the target: an element stays while the mass ahead of it is short
            const u64 ahead_a = incl - local, ahead_b = ahead_a + ea;
            const uint32_t ka = __ballot_sync(0xFFFFFFFFu, va && ahead_a < target);
            const uint32_t kb = __ballot_sync(0xFFFFFFFFu, vb && ahead_b < target);
            L8 = __popc(ka) + __popc(kb);
            const u64 through = ((L8 - 1) & 1) ? ahead_b + eb : ahead_b;     // mass through this lane's element of that parity
            S_fx = __shfl_sync(0xFFFFFFFFu, through, (L8 - 1) >> 1);
        }
        lnS = logf((float)(full_fx ? full_fx : S_fx) * (1.0f / FX_SCALE));
        tok = comp_idx(s0);
        lp_tok = full_fx ? __fsub_rn(unkey((uint32_t)(s0 >> 32)), zmax) - lnS : 0.0f;
        if (L8 > 1) {
            // argmax of the race score over the kept prefix (ties: lowest id, via the low word ~id)
            u64 best = 0, sbest = 0;
            if (qa < L8 && ga > best) { best = ga; sbest = sa; }
            if (qb < L8 && gb > best) { best = gb; sbest = sb; }
            const uint32_t ghi = __reduce_max_sync(0xFFFFFFFFu, (uint32_t)(best >> 32));
            const uint32_t glo = __reduce_max_sync(0xFFFFFFFFu, (uint32_t)(best >> 32) == ghi ? (uint32_t)best : 0u);
            const uint32_t who = __ballot_sync(0xFFFFFFFFu, (uint32_t)(best >> 32) == ghi && (uint32_t)best == glo);
            const u64 sw = __shfl_sync(0xFFFFFFFFu, sbest, __ffs(who) - 1);
            tok = comp_idx(sw);
            lp_tok = __fsub_rn(unkey((uint32_t)(sw >> 32)), zmax) - lnS;
        }
    } else {
    // Each lane owns a contiguous run of the sorted list.  Masses are fixed point: integer sums are
    // exact, so the prefix sums do not depend on the order of the additions.
    const int per = (L7 + 31) >> 5;
    const int q0 = lane * per, q1 = min(L7, q0 + per);
    u64 local = 0;
    for (int q = q0; q < q1; ++q) local += efx[q];
    u64 incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { u64 t2 = __shfl_up_sync(0xFFFFFFFFu, incl, o); if (lane >= o) incl += t2; }
    const u64 tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
    L8 = L7;
    u64 S_fx = tot;
    if (!rp.greedy && rp.top_p < 1.0f) {
        double t = ceil((double)rp.top_p * (double)tot);
        u64 target = t <= 1.0 ? 1ull : (u64)t;
        if (target > tot) target = tot;
        // smallest prefix whose mass reaches the target: keep an element while the mass ahead of it is short
        u64 run = incl - local, last = 0;
        int cnt = 0;
        for (int q = q0; q < q1; ++q) {
            const bool keep = run < target;
            run += efx[q];
            if (keep) { ++cnt; last = run; }
        }
        L8 = __reduce_add_sync(0xFFFFFFFFu, cnt);
        S_fx = __shfl_sync(0xFFFFFFFFu, last, (L8 - 1) / per);
    }
    lnS = logf((float)(full_fx ? full_fx : S_fx) * (1.0f / FX_SCALE));
    tok = comp_idx(sorted[0]);
    lp_tok = full_fx ? __fsub_rn(unkey((uint32_t)(sorted[0] >> 32)), zmax) - lnS : 0.0f;
    if (L8 > 1) {
        // argmax of the race score over the kept prefix (ties: lowest id, via the low word ~id)
        u64 best = 0; int bestq = 0;
        for (int q = q0; q < min(q1, L8); ++q) { u64 G = gsc[q]; if (G > best) { best = G; bestq = q; } }
        const uint32_t ghi = __reduce_max_sync(0xFFFFFFFFu, (uint32_t)(best >> 32));
        const uint32_t glo = __reduce_max_sync(0xFFFFFFFFu, (uint32_t)(best >> 32) == ghi ? (uint32_t)best : 0u);
        const uint32_t who = __ballot_sync(0xFFFFFFFFu, (uint32_t)(best >> 32) == ghi && (uint32_t)best == glo);
        const int wq = __shfl_sync(0xFFFFFFFFu, bestq, __ffs(who) - 1);
        tok = comp_idx(sorted[wq]);
        lp_tok = __fsub_rn(unkey((uint32_t)(sorted[wq] >> 32)), zmax) - lnS;
    }
    }
    out.token = tok; out.logprob = lp_tok; out.n_keep = L8;
    if (a.num_top > 0) {
        for (int q = lane; q < a.num_top && q < L8; q += 32) {
            const int64_t o = (int64_t)b * a.num_top + q;
            a.out_top_ids[o] = comp_idx(sorted[q]);
            a.out_top_logprobs[o] = (L8 == 1 && !full_fx) ? 0.0f : __fsub_rn(unkey((uint32_t)(sorted[q] >> 32)), zmax) - lnS;
        }
    }
}

// Threshold of the warm-up: a lower bound of the k-th largest of the block's per-thread maxima `mk`
// (0: the thread has none), all of which lie in [kmin, kmax].  One pass: the maxima fall into
// SEL_BINS value-linear bins (a monotone map of the key), each bin also keeps its smallest key; one
// warp then finds the bin in which the count from the top reaches k and the answer is that bin's
// smallest key: at least k maxima are not below it.  Returns 0 if there are fewer than k maxima.
// Needs cs.hist zero and the bin minima 0xFFFFFFFF on entry; contains two barriers, the last at the end.
__device__ uint32_t warm_select(BlockScratch &s, const CandSmem &cs, uint32_t mk, int k, uint32_t kmin, uint32_t kmax) {
    uint32_t *binmin = (uint32_t *)(cs.cand + SEL_BINS);
    const float zmin = unkey(kmin), d = unkey(kmax) - zmin;
    const float scale = (d > 0.0f && d <= 3.0e38f) ? __fdividef((float)(SEL_BINS - 1), d) : 0.0f;
    if (mk) {
        int q = (int)((unkey(mk) - zmin) * scale);
        q = q < 0 ? 0 : (q > SEL_BINS - 1 ? SEL_BINS - 1 : q);
        atomicAdd(&cs.hist[q], 1u);
        atomicMin(&binmin[q], mk);
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        constexpr int PER = SEL_BINS / 32;                 // consecutive bins per lane
        uint32_t cn[PER], sum = 0;
#pragma unroll
        for (int q = 0; q < PER; q += 4) {
            const uint4 v = *(const uint4 *)(cs.hist + PER * lane + q);
            cn[q] = v.x; cn[q + 1] = v.y; cn[q + 2] = v.z; cn[q + 3] = v.w;
            sum += v.x + v.y + v.z + v.w;
        }
        uint32_t suf = sum;                                // maxima in this lane's bins and above
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const uint32_t t = __shfl_down_sync(0xFFFFFFFFu, suf, o); if (lane + o < 32) suf += t; }
        uint32_t above = suf - sum;
        if (lane == 0 && suf < (uint32_t)k) s.found_digit = 0u;
        if (above < (uint32_t)k && suf >= (uint32_t)k) {   // exactly one lane
            int q = PER - 1;
#pragma unroll
            for (int j = PER - 1; j > 0; --j) { if (above + cn[j] < (uint32_t)k && q == j) { above += cn[j]; q = j - 1; } }
            s.found_digit = binmin[PER * lane + q];
        }
    }
    __syncthreads();
    return s.found_digit;
}

// Starts the stream of a row: resets the per-row state, arms the mbarriers and issues the first
// copies.  Called first thing in the kernel, before the row's parameters are loaded and the history
// tables built, so that the first tiles arrive meanwhile; a block barrier must follow before any wait.
// The ring's barriers and the block's bookkeeping: touches shared memory only, so under programmatic
// dependent launch it runs before the wait for the kernel ahead (thread 0 only).
__device__ __forceinline__ void ring_setup(BlockScratch &s, const Ring &rg) {
    if (threadIdx.x != 0) return;
    for (int st = 0; st < rg.nstages; ++st) mbar_init(&rg.bar[st], 1);
    mbar_init(&rg.bar[MAX_STAGES - 1], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    s.cand_cnt = 0; s.overflow = 0; s.runmax = 0; s.timeout = 0; s.issued = 0;
    s.mm_max = 0; s.mm_min = 0xFFFFFFFFu; s.found_digit = 0xFFFFFFFFu; s.maint_at = 0xFFFFFFFFu;
    for (int q = 0; q < MAX_STAGES; ++q) s.done[q] = 0;
}
// The first copies of the row (thread 0 only; after ring_setup).
template <int DT>
__device__ void candidate_begin(BlockScratch &s, const Ring &rg, const RowCtx &c) {
    typedef Elem<DT> E;
    if (threadIdx.x != 0) return;
    const uintptr_t addr = (uintptr_t)c.row;
    int head = (int)(((16u - (uint32_t)(addr & 15u)) & 15u) / E::SIZE);
    if (head > c.V) head = c.V;
    const int nvec = (c.V - head) / E::PER_VEC;
    const uint4 *vp = (const uint4 *)((const char *)c.row + (size_t)head * E::SIZE);
    const int ntiles = (nvec + NT * TILE_VECS - 1) / (NT * TILE_VECS);
    if (ntiles > 0) ring_issue_first(rg, vp, nvec);
    const int npre = ntiles < rg.nstages ? ntiles : rg.nstages;
    for (int t = 1; t < npre; ++t) ring_issue(rg, vp, nvec, t, t);
    s.issued = (uint32_t)npre;
}

// which rows the candidate path takes (decided from the row's parameters alone)
// (a top-N list over the whole vocabulary is the general path's business: the candidate list ends
// where the cuts end)
__device__ __forceinline__ bool candidate_eligible(const RowParams &rp, int V, bool full_list) {
    if (full_list) return false;
    const int k = rp.greedy ? 1 : rp.top_k;
    const bool has_topk = rp.greedy || (k >= 1 && k < V);
    const bool has_minp = !rp.greedy && rp.min_p > 0.0f;
    if (has_topk && k > KA_MAX) return false;
    return has_topk || has_minp;
}

// Returns false if the row must be handled by the general path instead.  On success the
// results are in `out` for warp 0 only.
template <int DT>
__device__ bool candidate_path(BlockScratch &s, const CandSmem &cs, const Ring &rg, const RowCtx &c,
                               const RowParams &rp, const SampleArgs &a, int b, RowOut &out) {
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
    const int lane = threadIdx.x & 31;
    // Thread -> vector map inside each group of NT vectors: lane l of warp w takes vector
    // 16 l + ((w + l) & 15).  Consecutive vectors land in different warps (the head of the
    // vocabulary, where large logits cluster, is shared by all warps) and the 16-byte shared
    // memory reads of a quarter warp still fall in distinct bank groups.
    const int pvec = 16 * lane + (((threadIdx.x >> 5) + lane) & 15);

    const uintptr_t addr = (uintptr_t)c.row;
    int head = (int)(((16u - (uint32_t)(addr & 15u)) & 15u) / E::SIZE);
    if (head > V) head = V;
    const int nvec = (V - head) / E::PER_VEC;
    const uint4 *vp = (const uint4 *)((const char *)c.row + (size_t)head * E::SIZE);
    const int ntiles = (nvec + NT * TILE_VECS - 1) / (NT * TILE_VECS);

    cs.hist[threadIdx.x] = 0;
    ((uint32_t *)(cs.cand + SEL_BINS))[threadIdx.x] = 0xFFFFFFFFu;     // warm_select's bin minima
    __syncthreads();

    uint32_t tau_topk = KEY_MIN_FINITE;   // the top-k part of the threshold: identical in every thread
    uint32_t tau_key = KEY_MIN_FINITE;    // the threshold in use: max(tau_topk, min-p floor this warp has seen)
    uint32_t thr = 0;
    uint32_t seen_max = 0;
    const uint32_t trig0 = has_topk ? (uint32_t)min(CAND_CAP / 2, 4 * k + 64) : (uint32_t)(CAND_CAP / 2);
    uint32_t trig = trig0;

    if (ntiles > 0) {
        // warm-up on the first NT vectors: the k-th largest of the per-thread maxima (each an
        // unpenalised element of the row, all distinct) is a lower bound of the row's k-th
        // largest score
        // (a large k needs a larger sample to give a useful bound: then the whole first tile; so do
        // fp32 rows, whose vectors hold half as many elements, and short rows, which have few tiles
        // over which a loose bound could still be tightened)
        const int wvecs = (has_topk && (k > 64 || E::PER_VEC < 8 || ntiles <= 6)) ? TILE_VECS : 1;
        bool bad = !mbar_wait(&rg.bar[MAX_STAGES - 1], 0);
        if (wvecs > 1 && !bad) bad = !mbar_wait(&rg.bar[0], 0);
        uint32_t mk = 0;
        for (int u = 0; u < wvecs; ++u) {
            const int v = u * NT + pvec;
            if (v < nvec && !bad) {
                const uint4 q = ((const uint4 *)rg.buf)[v];
                const int i0 = head + v * E::PER_VEC;
                uint32_t kk;
                if (c.has_hist && (__funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31) & ((1u << E::PER_VEC) - 1u)))
                    kk = masked_vmax_key<DT>(c, q, i0);
                else
                    kk = T::vmax_key(q, c.invT);
                mk = kk > mk ? kk : mk;
            }
        }
        if (mk < KEY_MIN_FINITE || mk >= KEY_POS_INF) mk = 0;
        {
            const uint32_t wmx = __reduce_max_sync(0xFFFFFFFFu, mk);
            const uint32_t wmn = __reduce_min_sync(0xFFFFFFFFu, mk ? mk : 0xFFFFFFFFu);
            if (lane == 0 && wmx) { atomicMax(&s.mm_max, wmx); atomicMin(&s.mm_min, wmn); }
        }
        if (bad) s.timeout = 1u;
        __syncthreads();
        const uint32_t kmax = s.mm_max, kmin = s.mm_min;
        if (stream_minp && threadIdx.x == 0) s.runmax = kmax;
        // fewer than k valid maxima: the select fails and tau stays at its floor
        if (has_topk && kmax) {
            const uint32_t t = warm_select(s, cs, mk, k, kmin, kmax);
            if (t > tau_topk) tau_topk = t;
        }
        tau_key = tau_topk;
        if (stream_minp && kmax) { uint32_t f = minp_key(unkey(kmax), rp.ln_min_p); tau_key = f > tau_key ? f : tau_key; }
        seen_max = kmax;
        thr = T::raw_threshold(tau_key, c.invT);
        if (!(has_topk && kmax)) __syncthreads();       // (the select ends with a barrier of its own)
    }

    // The consumer warps run decoupled: no block barrier per tile.  A stage is refilled by the
    // last warp that finishes with it.  Block-wide work on the candidate list (tightening the
    // threshold, overflow, expired waits) happens at a rendezvous: a warp working on tile t asks
    // for one before tile t + nstages + 1.  No warp can have looked at that boundary yet: it is
    // reached only after tile t + nstages, whose data is requested only when every warp is done
    // with tile t.  Every warp checks s.maint_at before each tile.
    int st = 0;                      // ring stage of the current tile
    uint32_t parity = 0;             // its mbarrier phase
    const bool early_ckpt = ntiles <= rg.nstages + 2;
    const uint32_t low_trig = (uint32_t)(has_topk ? 2 * k + 32 : CAND_CAP / 4);
    bool first_look = true;
    for (int tile = 0; tile < ntiles; ++tile) {
        // Tile 0 holds the head of the vocabulary and is the densest, and a bound from 4x the warm-up
        // sample is much tighter: if the list is already long after it, it is looked at early --
        // in short rows at a fixed checkpoint before tile 1, in long rows at a rendezvous that the
        // last warp to finish tile 0 asks for (see below), which costs rows with a short list nothing.
        if ((uint32_t)tile == *(volatile uint32_t *)&s.maint_at || (early_ckpt && tile == 1)) {
            __syncthreads();                       // every warp is between tiles: nobody appends
            int n = (int)s.cand_cnt;
            const uint32_t ovf = s.overflow, rmax = s.runmax, tmo = s.timeout;
            __syncthreads();
            if (threadIdx.x == 0 && (uint32_t)tile == s.maint_at) s.maint_at = 0xFFFFFFFFu;
            if (ovf || tmo) {
                ring_drain(rg, max(0, (int)s.issued - rg.nstages), (int)s.issued);
                if (tmo) { out.status |= ALBIREO_ROW_TIMEOUT; out.token = -1; out.logprob = __uint_as_float(0x7FC00000u); out.n_keep = 0; out.n_topk = 0; return true; }
                __syncthreads();
                return false;
            }
            // make the threshold identical in every thread again
            uint32_t tau_new = tau_topk;
            if (stream_minp && rmax) { seen_max = rmax; uint32_t f = minp_key(unkey(rmax), rp.ln_min_p); tau_new = f > tau_new ? f : tau_new; }
            const uint32_t trig_now = first_look ? min(trig, low_trig) : trig;
            first_look = false;
            if ((uint32_t)n + 1u >= trig_now) {
                if (has_topk && n >= k) {
                    uint32_t t = cand_select_approx(s, cs, n, k, tau_topk, rmax);
                    if (t > tau_topk) tau_topk = t;
                    if (t > tau_new) tau_new = t;
                }
                n = cand_compact(s, cs, n, tau_new);
                // if the list could not be shrunk (ties), look again only after it has grown
                trig = (uint32_t)n + (uint32_t)(has_topk ? 2 * k + 32 : CAND_CAP / 4);
                if (trig < trig0) trig = trig0;
            }
            if (tau_new != tau_key) { tau_key = tau_new; thr = T::raw_threshold(tau_key, c.invT); }
            __syncthreads();                       // s.maint_at is reset before anyone asks again
        }
        if (stream_minp) {
            // the min-p floor follows the running maximum without any block-wide step: a warp that
            // still uses an older (lower) floor is merely less selective
            const uint32_t rm = *(volatile uint32_t *)&s.runmax;
            if (rm > seen_max) {
                seen_max = rm;
                const uint32_t f = minp_key(unkey(rm), rp.ln_min_p);
                if (f > tau_key) { tau_key = f; thr = T::raw_threshold(tau_key, c.invT); }
            }
        }
        const int vbase = tile * NT * TILE_VECS;
        bool ask = false;                          // ask for a rendezvous
        const bool dead = *(volatile uint32_t *)&s.timeout != 0u;   // a wait expired somewhere: only keep the protocol going
        if (!dead) {
            if (!mbar_wait(&rg.bar[st], parity)) { s.timeout = 1u; ask = true; }
            else {
                const uint4 *stage = (const uint4 *)(rg.buf + (size_t)st * STAGE_BYTES) + pvec;
                uint4 cur[TILE_VECS];
                if (vbase + NT * TILE_VECS <= nvec) {
#pragma unroll
                    for (int u = 0; u < TILE_VECS; ++u) cur[u] = stage[u * NT];
                } else {
#pragma unroll
                    for (int u = 0; u < TILE_VECS; ++u)
                        cur[u] = (vbase + u * NT + pvec < nvec) ? stage[u * NT] : T::fill();
                }
                // scan: one cheap test for this thread's share of the tile; the element test only in
                // warps where some vector may pass
                if (__any_sync(0xFFFFFFFFu, T::any_may_pass(cur, thr, c.invT))) {
                    // per-element test in the test domain (a superset of key >= tau), minus penalised tokens
                    uint32_t all = 0;
#pragma unroll
                    for (int u = 0; u < TILE_VECS; ++u) {
                        uint32_t bts = T::elem_bits(cur[u], thr, c.invT);
                        if (c.has_hist && bts) {
                            const int i0 = head + (vbase + u * NT + pvec) * E::PER_VEC;
                            bts &= ~__funnelshift_r(c.bitmap[i0 >> 5], c.bitmap[(i0 >> 5) + 1], i0 & 31);
                        }
                        all |= bts << (u * E::PER_VEC);
                    }
                    const uint32_t cnt = __popc(all);
                    if (__any_sync(0xFFFFFFFFu, cnt != 0)) {
                        // one reservation per warp, then every lane writes its survivors (re-read from the stage)
                        const uint32_t inc = warp_incl_scan_u32(cnt);
                        const uint32_t total = __shfl_sync(0xFFFFFFFFu, inc, 31);
                        uint32_t base = 0;
                        if (lane == 31) base = atomicAdd(&s.cand_cnt, total);
                        base = __shfl_sync(0xFFFFFFFFu, base, 31);
                        ask = base + total + 1u >= trig;
                        if (base + total > (uint32_t)CAND_CAP) { if (lane == 31) s.overflow = 1u; ask = true; }
                        else {
                            uint32_t slot = base + inc - cnt;
                            uint32_t lmax = 0;
                            while (all) {
                                const int pbit = __ffs(all) - 1;
                                all &= all - 1;
                                const int u = pbit / E::PER_VEC, e = pbit % E::PER_VEC;
                                const float x = E::load_plain((const void *)(stage + u * NT), e);
                                const uint32_t key = key_of(__fmul_rn(x, c.invT));
                                cs.cand[slot++] = comp_of(key, head + (vbase + u * NT + pvec) * E::PER_VEC + e);
                                lmax = key > lmax ? key : lmax;
                            }
                            lmax = __reduce_max_sync(0xFFFFFFFFu, lmax);
                            if (lane == 0 && lmax > *(volatile uint32_t *)&s.runmax) {
                                const uint32_t old = atomicMax(&s.runmax, lmax);
                                (void)old;
                            }

                        }
                    }
                }
            }
        }
        if (__any_sync(0xFFFFFFFFu, ask) && lane == 0) atomicMin(&s.maint_at, (uint32_t)(tile + rg.nstages + 1));
        __syncwarp();
        if (lane == 0) {
            __threadfence_block();                 // this warp's reads of the stage come before its arrival
            const uint32_t old = atomicAdd(&s.done[st], 1u);
            if (old == (uint32_t)(NWARPS - 1)) {   // last warp done with this stage: refill it
                s.done[st] = 0;
                __threadfence_block();
                // every warp has finished tile 0 and none can be past tile nstages (not loaded yet):
                // a long list is looked at before tile nstages + 1
                if (tile == 0 && !early_ckpt && *(volatile uint32_t *)&s.cand_cnt + 1u >= low_trig)
                    atomicMin(&s.maint_at, (uint32_t)(rg.nstages + 1));
                if (tile + rg.nstages < ntiles && *(volatile uint32_t *)&s.timeout == 0u) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    ring_issue(rg, vp, nvec, tile + rg.nstages, st);
                    atomicMax(&s.issued, (uint32_t)(tile + rg.nstages + 1));
                }
            }
        }
        if (++st == rg.nstages) { st = 0; parity ^= 1u; }
    }
    // No barrier here: a warp that has left the loop only appends (atomic slots, its own threshold),
    // like the warps still streaming, and no rendezvous can be pending that it has not attended.
    // scalar head and tail of a row that is not 16-byte aligned / not a whole number of vectors
    {
        const int tail0 = head + nvec * E::PER_VEC;
        const int nscal = head + (V - tail0);
        for (int q = threadIdx.x; q < nscal; q += NT) {
            int i = q < head ? q : tail0 + (q - head);
            if (c.has_hist && ((c.bitmap[i >> 5] >> (i & 31)) & 1u)) continue;
            uint32_t key = key_of(__fmul_rn(E::load(elem_ptr<DT>(c, i), 0), c.invT));
            if (key >= tau_key) cand_append_one(s, cs, comp_of(key, i));
        }
    }
    // penalised tokens, straight from the history tables: one distinct id per thread and round,
    // so that a dense head of the vocabulary does not pile up on a few threads; four rounds at a
    // time, so that their scattered loads (a round trip each, behind the other rows' streams) overlap
    if (c.has_hist) {
        constexpr int PG = 4;
        for (uint32_t r0 = threadIdx.x; r0 < c.n_distinct; r0 += PG * NT) {
            int id[PG]; float x[PG];
#pragma unroll
            for (int u = 0; u < PG; ++u) { const uint32_t r = r0 + u * NT; id[u] = r < c.n_distinct ? hist_id_of_rank(c, r) : -1; }
#pragma unroll
            for (int u = 0; u < PG; ++u) x[u] = id[u] >= 0 ? E::load(elem_ptr<DT>(c, id[u]), 0) : 0.0f;
#pragma unroll
            for (int u = 0; u < PG; ++u) {
                if (id[u] < 0) continue;
                const float av = penalise_counted(c, x[u], c.counts[r0 + u * NT]);
                const uint32_t key = key_of(__fmul_rn(av, c.invT));
                if (key >= tau_key) cand_append_one(s, cs, comp_of(key, id[u]));
            }
        }
    }
    __syncthreads();
    int n = (int)s.cand_cnt;
    const uint32_t ovf = s.overflow, tmo_end = s.timeout;
    // (no second barrier: nothing below writes these words before a barrier of its own -- the
    // compaction's -- that every thread reaches only after it has read them here)
    if (tmo_end) {
        ring_drain(rg, max(0, (int)s.issued - rg.nstages), (int)s.issued);
        out.status |= ALBIREO_ROW_TIMEOUT; out.token = -1; out.logprob = __uint_as_float(0x7FC00000u); out.n_keep = 0; out.n_topk = 0;
        return true;
    }
    if (ovf || n < 1) return false;

    const uint32_t kmax = s.runmax;    // the row's largest score is always a candidate
    bool topk_exact_known = true;      // is min(k, #finite) known without counting?
    // keep-ties mode: the top-k stage keeps every score not below the k-th largest, i.e. exactly the
    // candidates that are left once the list is cut at the k-th largest key
    const bool keep_ties = has_topk && !rp.greedy && (a.flags & ALBIREO_FLAG_TOPK_KEEP_TIES);
    if (has_topk) {
        if (n > SORT_MAX || n > 2 * k + 96 || (keep_ties && n > k)) {
            uint32_t t = cand_select_exact(s, cs, n, k, tau_key, kmax);
            n = cand_compact(s, cs, n, t);
        }
        if (n < k && stream_minp) topk_exact_known = false;
    } else {
        n = cand_compact(s, cs, n, minp_key(unkey(kmax), rp.ln_min_p));
        topk_exact_known = false;
    }
    if (n > SORT_MAX || n < 1) return false;

    const int L6 = has_topk ? ((n < k || keep_ties) ? n : k) : n;
    int n_topk = L6;
    if (!topk_exact_known && a.out_num_topk) {
        // diagnostic only: count the finite scores of the row
        uint32_t local = 0;
        for_each_score<DT>(c, [&](int, float z) { uint32_t kk = key_of(z); local += (kk >= KEY_MIN_FINITE && kk < KEY_POS_INF); });
        u64 nfin = block_sum_u64(s, local);
        n_topk = has_topk ? (int)(nfin < (u64)k ? nfin : (u64)k) : (int)nfin;
    }
    out.n_topk = n_topk;
    const u64 full_fx = (a.flags & ALBIREO_FLAG_LOGPROB_FULL_VOCAB) ? full_vocab_mass<DT>(s, c, unkey(kmax)) : 0ull;
    // the stream is over: a dependent kernel launched the same way may be scheduled from here on
    if (a.flags & ALBIREO_FLAG_PROGRAMMATIC_LAUNCH) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    final_stage(s, cs, n, L6, unkey(kmax), has_minp, rp, a, b, out, full_fx);
    return true;
}

// ------------------------------------------------------------------ the kernel

// dynamic shared memory layout (bytes): [candidates (8 KiB) + 512 select bins (2 KiB)]
// [ring: nstages x 32 KiB][mbarriers][bitmap][coarse][counts]; the general path lays its histograms,
// gather list and search bins (8 + 24 + 16 + 4 KiB) over the first 52 KiB, which it may do because
// the ring is idle by then
template <int DT>
__global__ void __launch_bounds__(NT, 2) albireo_sample_kernel(const SampleArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ BlockScratch s;
    const int b = blockIdx.x;
    const int V = a.V;

    Ring rg;
    rg.nstages = a.nstages;
    rg.vps = a.vps;
    rg.seg_base = s.seg_base;
    rg.buf = smem + COMMON_BYTES;
    rg.bar = (uint64_t *)(rg.buf + (size_t)a.nstages * STAGE_BYTES);
    // A row that turns out to need the general path waits for the ring's copies before it reuses the
    // shared memory.
    const bool ring_started = !(a.flags & ALBIREO_FLAG_FORCE_GENERAL);
    if (ring_started) ring_setup(s, rg);
    // Under programmatic dependent launch the CTA may have been scheduled while the kernel ahead in the
    // stream (the producer of the logits) was still running: everything above touched only launch
    // arguments and shared memory; nothing below is read or written before that kernel has finished.
    if (a.flags & ALBIREO_FLAG_PROGRAMMATIC_LAUNCH) asm volatile("griddepcontrol.wait;" ::: "memory");
    // The row's own parameters and the first part of its history are asked for before the ring is started: a
    // load issued after the ring's copies (this CTA's and every other's) queues behind megabytes of
    // them; issued before, it is back within an idle round trip, while thread 0 is still setting up.
    // With histories the loads come first (the history build waits for them, and so does every thread
    // at its first barrier); without, they follow the ring start as the first tiles travel, since
    // reading a dozen more launch arguments first would hold the ring back for nothing.
    RowParams rp;
    RowCtx c;
    int o0 = 0, o1 = 0, ostart = 0;
    const bool with_hist = a.hist_ids && a.hist_off;
    auto load_params = [&]() {
        rp.T = a.temperature ? a.temperature[b] : 1.0f;
        rp.top_k = a.top_k ? a.top_k[b] : 0;
        rp.top_p = a.top_p ? a.top_p[b] : 1.0f;
        rp.min_p = a.min_p ? a.min_p[b] : 0.0f;
        rp.seed = a.seeds ? a.seeds[b] : 0ull;
        c.r = a.rep ? a.rep[b] : 1.0f;
        c.p = a.pres ? a.pres[b] : 0.0f;
        c.f = a.freq ? a.freq[b] : 0.0f;
    };
    rp.R = a.row_base + (uint32_t)b;
    if (with_hist) {
        load_params();
        o0 = a.hist_off[b]; o1 = a.hist_off[b + 1];
        if (a.out_start) ostart = a.out_start[b];
        if (o1 > o0) hist_prefetch(a.hist_ids + o0, o1 - o0, (int32_t *)smem);
    }
    c.row = (const char *)a.logits + (size_t)b * (size_t)a.row_stride * Elem<DT>::SIZE;
    c.V = V;
    c.nseg = a.nseg; c.Vs = a.Vs; c.seg_base = s.seg_base;
    if (a.nseg > 1) {
        // where the pieces of this row start: a stride apart in one buffer, or one buffer per piece (the
        // senders' own memory, read in place over NVLink: then there is no exchange step at all)
        const size_t row_off = (size_t)(a.seg_row_offset + b) * (size_t)a.row_stride * Elem<DT>::SIZE;
        if (a.seg_ptr_count > 0) c.row = (const char *)a.seg_ptr[0] + row_off;
        if (threadIdx.x == 0) {             // thread 0 issues the ring's copies; everyone else reads the table after a barrier
            for (int j = 0; j < a.nseg; ++j)
                s.seg_base[j] = a.seg_ptr_count > 0 ? (const char *)a.seg_ptr[j] + row_off
                                                    : (const char *)c.row + (size_t)j * (size_t)a.seg_stride * Elem<DT>::SIZE;
        }
    }
    if (ring_started) candidate_begin<DT>(s, rg, c);
    if (!with_hist) load_params();

    HistSmem hs;
    const int nwords = (V + 31) >> 5, ncoarse = (nwords + 7) >> 3;
    hs.bitmap = (uint32_t *)((unsigned char *)rg.bar + MAX_STAGES * 8);
    hs.coarse = hs.bitmap + (nwords + 1);
    hs.counts = hs.coarse + (ncoarse + 1);

    rp.greedy = !(rp.T > 0.0f);
    rp.ln_min_p = (!rp.greedy && rp.min_p > 0.0f) ? log((double)rp.min_p) : 0.0;

    RowOut out;
    out.token = 0; out.logprob = 0.0f; out.n_keep = 0; out.n_topk = 0; out.status = 0;
    if (rp.T < 0.0f || rp.T != rp.T) out.status |= ALBIREO_ROW_BAD_PARAM;

    c.invT = rp.greedy ? 1.0f : __fdiv_rn(1.0f, rp.T);
    c.has_hist = false; c.bitmap = nullptr; c.coarse = nullptr; c.counts = nullptr; c.n_distinct = 0; c.ncoarse = 0;
    if (!(c.r > 0.0f)) out.status |= ALBIREO_ROW_BAD_PARAM;

    const bool try_candidates = ring_started && candidate_eligible(rp, V, (a.flags & ALBIREO_FLAG_LOGPROB_FULL_VOCAB) && a.num_top > 0);
    if (o1 > o0) {
        bool ok = build_history(s, hs, c, a.hist_ids + o0, o1 - o0, ostart, (const int32_t *)smem, a.ws_counts, a.ws_counts_cap, (int64_t)o0);
        c.has_hist = ok;
        if (!ok) out.status |= ALBIREO_ROW_HISTORY_OVERFLOW;
    }

    // dbg / top-N padding first, the paths overwrite what they produce
    if (a.dbg_topk_ids) for (int j = threadIdx.x; j < a.dbg_cap; j += NT) a.dbg_topk_ids[(int64_t)b * a.dbg_cap + j] = -1;
    if (a.num_top > 0) for (int j = threadIdx.x; j < a.num_top; j += NT) {
        a.out_top_ids[(int64_t)b * a.num_top + j] = -1;
        a.out_top_logprobs[(int64_t)b * a.num_top + j] = __uint_as_float(0xFF800000u);
    }
    __syncthreads();

    CandSmem cs;
    cs.cand = (u64 *)smem;                                  // 8 KiB
    cs.hist = (uint32_t *)(smem + CAND_CAP * 8);            // 2 KiB
    cs.sorted = (u64 *)rg.buf;                              // 3 x 4 KiB in the ring, used after the stream
    cs.efx = cs.sorted + SORT_MAX;
    cs.gsc = cs.efx + SORT_MAX;
    bool done = false;
    if (try_candidates) done = candidate_path<DT>(s, cs, rg, c, rp, a, b, out);
    else if (ring_started) {
        // (the barrier above made s.issued visible)
        bool landed = mbar_wait(&rg.bar[MAX_STAGES - 1], 0u);
        for (int t = 0; t < (int)s.issued; ++t) landed = mbar_wait(&rg.bar[t], 0u) && landed;
        if (__syncthreads_or(!landed)) { out.status |= ALBIREO_ROW_TIMEOUT; out.token = -1; out.logprob = __uint_as_float(0x7FC00000u); done = true; }   // the same in every thread
    }
    if (!done) {
        if (threadIdx.x == 0) {
            GenArgs &ga = s.ga;
            ga.dbg_topk_ids = a.dbg_topk_ids; ga.exp1 = a.exp1; ga.exp1_stride = a.exp1_stride; ga.out_top_ids = a.out_top_ids;
            ga.out_top_logprobs = a.out_top_logprobs; ga.step = a.step; ga.flags = a.flags; ga.num_top = a.num_top; ga.dbg_cap = a.dbg_cap;
        }
        __syncthreads();
        out = general_path_call<DT>(&s, smem, c, rp, b, out.status);
    }

    if (threadIdx.x == 0) {
        a.out_tokens[b] = out.token;
        a.out_logprobs[b] = out.logprob;
        if (a.out_num_kept) a.out_num_kept[b] = out.n_keep;
        if (a.out_num_topk) a.out_num_topk[b] = out.n_topk;
        // early feedback (section 5.2): the token goes straight into the next iteration's input ids
        // and to the output processor's ring, without waiting for a host round trip
        const bool have_token = !(out.status & ALBIREO_ROW_TIMEOUT);
        if (a.backfill_ids && have_token) {
            const int64_t slot = a.backfill_index ? (int64_t)a.backfill_index[b] : (int64_t)b;
            if (slot >= 0) {
                if (slot < a.backfill_len) a.backfill_ids[slot] = out.token;
                else out.status |= ALBIREO_ROW_BAD_PARAM;
            }
        }
        if (a.feedback_ring && have_token) {
            const int64_t slot = (a.feedback_head + b) % a.feedback_cap;
            const unsigned long long rec = ((unsigned long long)(a.row_base + (uint32_t)b) << 32) | (uint32_t)out.token;
            *(volatile unsigned long long *)(a.feedback_ring + slot) = rec;      // one 8-byte store
        }
        if (a.out_row_status) a.out_row_status[b] = out.status;
    }
}

// ------------------------------------------------------------------ the stream alone (measurement aid)
//
// The same ring, the same launch shape (a CTA per row, 512 threads, two CTAs per SM), the same
// packed test of every tile against a threshold nothing reaches -- and nothing else: no threshold to
// set up, no candidates, no final stage.  What this kernel takes is what the stream itself costs on
// this GPU at this size; the sampler's own work is the difference.  Writes one word per row so that
// the loads cannot be dropped.
template <int DT>
__global__ void __launch_bounds__(NT, 2) albireo_stream_only_kernel(const void *logits, int V, int64_t row_stride, int nstages, uint32_t *sink, int drop_tile) {
    typedef Elem<DT> E;
    typedef VecTest<DT> T;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ uint32_t done[MAX_STAGES];
    __shared__ uint32_t hits, dead, issued;
    __shared__ const char *no_pieces[1];
    Ring rg;
    rg.nstages = nstages; rg.vps = 0x7FFFFFFF; rg.seg_base = no_pieces;
    rg.buf = smem + COMMON_BYTES;
    rg.bar = (uint64_t *)(rg.buf + (size_t)nstages * STAGE_BYTES);
    const char *row = (const char *)logits + (size_t)blockIdx.x * (size_t)row_stride * E::SIZE;
    int head = (int)(((16u - (uint32_t)((uintptr_t)row & 15u)) & 15u) / E::SIZE);
    if (head > V) head = V;
    const int nvec = (V - head) / E::PER_VEC;
    const uint4 *vp = (const uint4 *)(row + (size_t)head * E::SIZE);
    const int ntiles = (nvec + NT * TILE_VECS - 1) / (NT * TILE_VECS);
    if (threadIdx.x == 0) {
        for (int st = 0; st < nstages; ++st) { mbar_init(&rg.bar[st], 1); done[st] = 0; }
        hits = 0; dead = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const int npre = ntiles < nstages ? ntiles : nstages;
        for (int t = 0; t < npre; ++t) {
            if (t == drop_tile) mbar_expect_tx(&rg.bar[t], 16u);      // announced, never copied: the wait on it must expire
            else ring_issue(rg, vp, nvec, t, t);
        }
        issued = (uint32_t)npre;
    }
    __syncthreads();
    // with a tile withheld the wait is meant to expire: a smaller bound keeps that launch short
    const int wait_cap = drop_tile >= 0 ? (1 << 14) : WAIT_CAP;
    const int lane = threadIdx.x & 31;
    const int pvec = 16 * lane + (((threadIdx.x >> 5) + lane) & 15);
    const uint32_t thr = T::pos_inf_threshold();      // only +inf reaches it
    int st = 0; uint32_t parity = 0, cnt = 0;
    for (int tile = 0; tile < ntiles; ++tile) {
        if (*(volatile uint32_t *)&dead == 0u) {
            if (!mbar_wait(&rg.bar[st], parity, wait_cap)) dead = 1u;        // (bounded: the row is given up, the protocol below goes on)
            else {
                const uint4 *stage = (const uint4 *)(rg.buf + (size_t)st * STAGE_BYTES) + pvec;
                const int vbase = tile * NT * TILE_VECS;
                uint4 cur[TILE_VECS];
#pragma unroll
                for (int u = 0; u < TILE_VECS; ++u) cur[u] = (vbase + u * NT + pvec < nvec) ? stage[u * NT] : T::fill();
                if (__any_sync(0xFFFFFFFFu, T::any_may_pass(cur, thr, 1.0f))) cnt += 1;
            }
        }
        __syncwarp();
        if (lane == 0) {
            __threadfence_block();
            const uint32_t old = atomicAdd(&done[st], 1u);
            if (old == (uint32_t)(NWARPS - 1)) {
                done[st] = 0;
                __threadfence_block();
                if (tile + nstages < ntiles && *(volatile uint32_t *)&dead == 0u) {
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    if (tile + nstages == drop_tile) mbar_expect_tx(&rg.bar[st], 16u);
                    else ring_issue(rg, vp, nvec, tile + nstages, st);
                    issued = (uint32_t)(tile + nstages + 1);
                }
            }
        }
        if (++st == nstages) { st = 0; parity ^= 1u; }
    }
    if (cnt && lane == 0) atomicAdd(&hits, cnt);
    __syncthreads();
    if (dead && threadIdx.x == 0) {
        // a wait expired: the copies still in flight land (bounded waits) before the CTA leaves
        const int hi = (int)issued, lo = hi - nstages > 0 ? hi - nstages : 0;
        for (int t = lo; t < hi; ++t) if (t != drop_tile) mbar_wait(&rg.bar[t % nstages], (uint32_t)(t / nstages) & 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) sink[blockIdx.x] = hits + (dead << 31);
}

size_t history_smem_bytes(int V) {
    size_t nwords = ((size_t)V + 31) / 32, ncoarse = (nwords + 7) / 8;
    return (nwords + 1 + ncoarse + 1 + CNT_CAP) * 4;
}
// ring depth: as deep as lets two CTAs share an SM (228 KiB per SM, 1 KiB reserved per CTA) -- or, for a
// batch with no more rows than the device has SMs (`alone`: every CTA has an SM to itself), as deep as
// one CTA's share allows
int ring_stages_for(int V, bool with_history, bool alone) {
    const long budget = (alone ? 233472 - 1024 : 233472 / 2 - 1024) - 1024;      // per CTA: dynamic bytes available
    long fixed = COMMON_BYTES + MAX_STAGES * 8 + (with_history ? (long)history_smem_bytes(V) : 0);
    long n = (budget - fixed) / STAGE_BYTES;
    const long cap = alone ? 6 : 4;
    if (n < 2) n = 2;
    if (n > cap) n = cap;
    return (int)n;
}
size_t smem_bytes_for(int V, bool with_history, int nstages) {
    size_t bytes = (size_t)COMMON_BYTES + (size_t)nstages * STAGE_BYTES + MAX_STAGES * 8;
    if (with_history) bytes += history_smem_bytes(V);
    return (bytes + 127) & ~(size_t)127;
}

constexpr size_t WS_HEADER = 256;

// Checks the optional arguments and copies them into the launch arguments; on failure *why says what.
int apply_ext(SampleArgs &a, const albireo_sample_ext_t *ext, int B, int V, const char **why) {
    (void)B;
    if (ext->struct_size != sizeof(albireo_sample_ext_t)) { *why = "ext->struct_size mismatch"; return ALBIREO_EINVAL; }
    if (ext->row_stride_elems != 0) {
        if (ext->row_stride_elems < V && ext->num_segments <= 1) { *why = "row stride smaller than V"; return ALBIREO_EINVAL; }
        a.row_stride = ext->row_stride_elems;
    }
    a.row_base = ext->row_base; a.flags = ext->flags;
    if (ext->num_top < 0 || ext->num_top > ALBIREO_MAX_NUM_TOP) { *why = "num_top out of range"; return ALBIREO_EUNSUPPORTED; }
    if (ext->num_top > 0 && (!ext->out_top_ids || !ext->out_top_logprobs)) { *why = "num_top > 0 needs both top-N outputs"; return ALBIREO_EINVAL; }
    a.num_top = ext->num_top; a.out_top_ids = ext->out_top_ids; a.out_top_logprobs = ext->out_top_logprobs;
    a.out_num_kept = ext->out_num_kept; a.out_num_topk = ext->out_num_topk;
    if (ext->dbg_cap < 0 || (ext->dbg_cap > 0 && !ext->dbg_topk_ids)) { *why = "bad dbg_cap / dbg_topk_ids"; return ALBIREO_EINVAL; }
    a.dbg_cap = ext->dbg_topk_ids ? ext->dbg_cap : 0;
    a.dbg_topk_ids = ext->dbg_cap > 0 ? ext->dbg_topk_ids : nullptr;
    a.out_row_status = ext->out_row_status;
    if (ext->num_segments > 1) {
        // rows in pieces: every piece must start and end on a 16-byte boundary
        const int64_t esz = a.elem_size, t = ext->num_segments;
        if (t > 64 || V % t) { *why = "num_segments must divide V and be at most 64"; return ALBIREO_EINVAL; }
        const int64_t Vs = V / t;
        if (!ext->segment_ptrs && ext->segment_stride_elems < Vs) { *why = "segment stride smaller than a piece"; return ALBIREO_EINVAL; }
        if (ext->row_stride_elems == 0) a.row_stride = Vs;
        if (a.row_stride < Vs) { *why = "row stride smaller than a piece"; return ALBIREO_EINVAL; }
        if ((Vs * esz) % 16 || (a.row_stride * esz) % 16 || (ext->segment_stride_elems * esz) % 16 || (uintptr_t)a.logits % 16) {
            *why = "rows in pieces need 16-byte aligned pieces, row stride, segment stride and base"; return ALBIREO_EUNSUPPORTED;
        }
        a.nseg = (int32_t)t; a.seg_stride = ext->segment_stride_elems;
        if (ext->segment_ptrs) {
            if (t > ALBIREO_MAX_PEER_SEGMENTS) { *why = "segment_ptrs takes at most ALBIREO_MAX_PEER_SEGMENTS pieces"; return ALBIREO_EUNSUPPORTED; }
            if (ext->segment_row_offset < 0) { *why = "segment_row_offset is negative"; return ALBIREO_EINVAL; }
            for (int64_t j = 0; j < t; ++j) {
                if (!ext->segment_ptrs[j] || (uintptr_t)ext->segment_ptrs[j] % 16) { *why = "segment_ptrs entries must be non-NULL and 16-byte aligned"; return ALBIREO_EUNSUPPORTED; }
                a.seg_ptr[j] = ext->segment_ptrs[j];
            }
            a.seg_ptr_count = (int32_t)t; a.seg_row_offset = ext->segment_row_offset;
        }
        a.Vs = (int32_t)Vs; a.vps = (int32_t)(Vs * esz / 16);
    } else if (ext->num_segments < 0) { *why = "num_segments is negative"; return ALBIREO_EINVAL; }
    a.out_start = ext->history_output_start;
    if (ext->exp1) {
        if (ext->exp1_stride_elems != 0 && ext->exp1_stride_elems < V) { *why = "exp1 row stride smaller than V"; return ALBIREO_EINVAL; }
        if ((uintptr_t)ext->exp1 % 4) { *why = "exp1 not 4-byte aligned"; return ALBIREO_EINVAL; }
        a.exp1 = ext->exp1; a.exp1_stride = ext->exp1_stride_elems ? ext->exp1_stride_elems : V;
    }
    if (ext->backfill_ids) {
        if (ext->backfill_len < 1) { *why = "backfill_ids needs backfill_len >= 1"; return ALBIREO_EINVAL; }
        a.backfill_ids = ext->backfill_ids; a.backfill_index = ext->backfill_index; a.backfill_len = ext->backfill_len;
    }
    if (ext->feedback_ring) {
        if (ext->feedback_cap < 1 || ext->feedback_head < 0) { *why = "feedback_ring needs feedback_cap >= 1 and feedback_head >= 0"; return ALBIREO_EINVAL; }
        if ((uintptr_t)ext->feedback_ring % 8) { *why = "feedback_ring not 8-byte aligned"; return ALBIREO_EINVAL; }
        a.feedback_ring = (unsigned long long *)ext->feedback_ring; a.feedback_cap = ext->feedback_cap;
        a.feedback_head = ext->feedback_head % ext->feedback_cap;
    }
    return ALBIREO_OK;
}

void launch_sample_kernel(int dtype, int B, size_t smem, cudaStream_t st, const SampleArgs &a) {
    if (a.flags & ALBIREO_FLAG_PROGRAMMATIC_LAUNCH) {
        // programmatic dependent launch: the kernel may be scheduled before the kernel ahead of it in the
        // stream has finished; it waits for that kernel itself (griddepcontrol.wait) before it touches memory
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)B); cfg.blockDim = dim3(NT); cfg.dynamicSmemBytes = smem; cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        if (dtype == ALBIREO_F32) cudaLaunchKernelEx(&cfg, albireo_sample_kernel<ALBIREO_F32>, a);
        else if (dtype == ALBIREO_BF16) cudaLaunchKernelEx(&cfg, albireo_sample_kernel<ALBIREO_BF16>, a);
        else cudaLaunchKernelEx(&cfg, albireo_sample_kernel<ALBIREO_F16>, a);
        return;
    }
    if (dtype == ALBIREO_F32) albireo_sample_kernel<ALBIREO_F32><<<B, NT, smem, st>>>(a);
    else if (dtype == ALBIREO_BF16) albireo_sample_kernel<ALBIREO_BF16><<<B, NT, smem, st>>>(a);
    else albireo_sample_kernel<ALBIREO_F16><<<B, NT, smem, st>>>(a);
}
// Lets every instantiation use the device's opt-in shared memory; gives the dynamic bytes available
// to a CTA (the opt-in limit less the largest static use), or 0 with *err set.
size_t enable_large_smem(int device, cudaError_t *err) {
    int optin = 0;
    cudaError_t e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    cudaFuncAttributes f0, f1, f2;
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&f0, albireo_sample_kernel<ALBIREO_F32>);
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&f1, albireo_sample_kernel<ALBIREO_BF16>);
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&f2, albireo_sample_kernel<ALBIREO_F16>);
    if (e != cudaSuccess) { *err = e; return 0; }
    size_t st = f0.sharedSizeBytes > f1.sharedSizeBytes ? f0.sharedSizeBytes : f1.sharedSizeBytes;
    if (f2.sharedSizeBytes > st) st = f2.sharedSizeBytes;
    if ((size_t)optin <= st) { *err = cudaErrorInvalidValue; return 0; }
    const size_t smem = (size_t)optin - st;
    e = cudaFuncSetAttribute(albireo_sample_kernel<ALBIREO_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(albireo_sample_kernel<ALBIREO_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(albireo_sample_kernel<ALBIREO_F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(albireo_stream_only_kernel<ALBIREO_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(albireo_stream_only_kernel<ALBIREO_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(albireo_stream_only_kernel<ALBIREO_F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    *err = e;
    return e == cudaSuccess ? smem : 0;
}

}  // namespace

// ------------------------------------------------------------------ C ABI

struct albireo_sampler {
    int32_t device;
    int32_t max_rows, max_vocab;
    int64_t max_history_total;
    unsigned char *workspace;
    size_t workspace_bytes;
    size_t max_smem;
    int num_sms;
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
    // opt in to the largest dynamic shared memory a CTA may have on this device
    cudaError_t e0 = cudaSuccess;
    const size_t smem = enable_large_smem(device, &e0);
    if (prev >= 0 && prev != device) cudaSetDevice(prev);
    if (e0 != cudaSuccess) { cudaGetLastError(); return ALBIREO_ECUDA; }
    if (smem_bytes_for(max_vocab, true, 2) > smem) return ALBIREO_EUNSUPPORTED;

    albireo_sampler *h = new (std::nothrow) albireo_sampler();
    if (!h) return ALBIREO_ENOMEM;
    h->device = device; h->max_rows = max_rows; h->max_vocab = max_vocab;
    h->max_history_total = max_history_total;
    h->workspace = (unsigned char *)workspace; h->workspace_bytes = workspace_bytes;
    h->max_smem = smem; h->launches = 0; h->err[0] = 0;
    h->num_sms = 0;
    if (cudaDeviceGetAttribute(&h->num_sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) { cudaGetLastError(); h->num_sms = 0; }
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
    if (dtype != ALBIREO_F32 && dtype != ALBIREO_BF16 && dtype != ALBIREO_F16) { set_err(h, "unknown dtype%s", ""); return ALBIREO_EINVAL; }
    if (!logits || !out_tokens || !out_logprobs) { set_err(h, "NULL logits or output%s", ""); return ALBIREO_EINVAL; }
    if ((history_ids == nullptr) != (history_offsets == nullptr)) { set_err(h, "history_ids and history_offsets must both be given%s", ""); return ALBIREO_EINVAL; }
    const size_t esize = dtype == ALBIREO_F32 ? 4 : 2;
    if ((uintptr_t)logits % esize) { set_err(h, "logits not element-aligned%s", ""); return ALBIREO_EINVAL; }

    SampleArgs a;
    memset(&a, 0, sizeof a);
    a.logits = logits; a.B = B; a.V = V; a.row_stride = V; a.nseg = 1; a.Vs = V; a.vps = 0x7FFFFFFF; a.elem_size = (int32_t)esize;
    a.temperature = temperature; a.top_k = top_k; a.top_p = top_p; a.min_p = min_p;
    a.rep = repetition_penalty; a.pres = presence_penalty; a.freq = frequency_penalty;
    a.hist_ids = history_ids; a.hist_off = history_offsets;
    a.seeds = seeds; a.step = step;
    a.out_tokens = out_tokens; a.out_logprobs = out_logprobs;
    a.ws_counts = (uint32_t *)(h->workspace + WS_HEADER);
    a.ws_counts_cap = h->max_history_total;
    if (ext) {
        const char *why = nullptr;
        const int rc = apply_ext(a, ext, B, V, &why);
        if (rc != ALBIREO_OK) { set_err(h, "%s", why); return rc; }
    }
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess || cur != h->device) { cudaGetLastError(); set_err(h, "the handle's device is not current%s", ""); return ALBIREO_EINVAL; }

    a.nstages = ring_stages_for(V, history_ids != nullptr, B <= h->num_sms);
    size_t smem = smem_bytes_for(V, history_ids != nullptr, a.nstages);
    while (smem > h->max_smem && a.nstages > 2) smem = smem_bytes_for(V, history_ids != nullptr, --a.nstages);
    if (smem > h->max_smem) { set_err(h, "vocabulary too large for the on-chip tables%s", ""); return ALBIREO_EUNSUPPORTED; }
    cudaStream_t st = (cudaStream_t)stream;
    launch_sample_kernel(dtype, B, smem, st, a);
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
    if (dtype != ALBIREO_F32 && dtype != ALBIREO_BF16 && dtype != ALBIREO_F16) { set_err(h, "unknown dtype%s", ""); return ALBIREO_EINVAL; }
    if (!logits || !out_tokens || !out_logprobs) { set_err(h, "NULL logits or output%s", ""); return ALBIREO_EINVAL; }
    if ((history_ids == nullptr) != (history_offsets == nullptr) || history_total < 0 || history_total > h->max_history_total) {
        set_err(h, "bad history arguments%s", ""); return ALBIREO_EINVAL;
    }
    if (ext && ext->struct_size != sizeof(albireo_sample_ext_t)) { set_err(h, "ext->struct_size mismatch%s", ""); return ALBIREO_EINVAL; }
    if (ext && ext->row_stride_elems != 0 && ext->row_stride_elems != V) { set_err(h, "host entry needs dense rows%s", ""); return ALBIREO_EINVAL; }
    if (ext && ext->dbg_cap > 0) { set_err(h, "host entry has no debug output%s", ""); return ALBIREO_EINVAL; }
    if (ext && (ext->num_top < 0 || ext->num_top > ALBIREO_MAX_NUM_TOP)) { set_err(h, "num_top out of range%s", ""); return ALBIREO_EUNSUPPORTED; }
    if (ext && (ext->exp1 || ext->backfill_ids || ext->feedback_ring || ext->num_segments > 1 || ext->history_output_start)) { set_err(h, "host entry takes no exp1 table, no early-feedback targets, no rows in pieces and no history split%s", ""); return ALBIREO_EINVAL; }
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

// Launches albireo_stream_only_kernel on the rows of `logits` (dense [B, V], one piece per row): see there.
extern "C" int albireo_stream_only(albireo_sampler_t *h, const void *logits, int32_t B, int32_t V, int32_t dtype,
                                   uint32_t *sink, int32_t drop_tile, void *stream) {
    if (!h) return ALBIREO_EINVAL;
    h->err[0] = 0;
    if (B == 0) return ALBIREO_OK;
    if (B < 0 || B > h->max_rows || V < 1 || V > h->max_vocab || !logits || !sink) { set_err(h, "bad arguments%s", ""); return ALBIREO_EINVAL; }
    if (dtype != ALBIREO_F32 && dtype != ALBIREO_BF16 && dtype != ALBIREO_F16) { set_err(h, "unknown dtype%s", ""); return ALBIREO_EINVAL; }
    int nstages = ring_stages_for(V, false, B <= h->num_sms);
    size_t smem = smem_bytes_for(V, false, nstages);
    while (smem > h->max_smem && nstages > 2) smem = smem_bytes_for(V, false, --nstages);
    if (smem > h->max_smem) { set_err(h, "vocabulary too large%s", ""); return ALBIREO_EUNSUPPORTED; }
    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == ALBIREO_F32) albireo_stream_only_kernel<ALBIREO_F32><<<B, NT, smem, st>>>(logits, V, (int64_t)V, nstages, sink, drop_tile);
    else if (dtype == ALBIREO_BF16) albireo_stream_only_kernel<ALBIREO_BF16><<<B, NT, smem, st>>>(logits, V, (int64_t)V, nstages, sink, drop_tile);
    else albireo_stream_only_kernel<ALBIREO_F16><<<B, NT, smem, st>>>(logits, V, (int64_t)V, nstages, sink, drop_tile);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) { set_err(h, "kernel launch failed: %s", cudaGetErrorString(e)); return ALBIREO_ECUDA; }
    return ALBIREO_OK;
}

// ------------------------------------------------------------------ entry point that allocates nothing
//
// Some callers cannot allocate device memory at the moment they need a sample: a plugin that
// runs inside a host whose memory pool is already fully handed out, a caller in the middle of
// work where cudaMalloc would synchronise the device, or code under a rule that forbids
// allocation after start-up.  For them the history-count scratch that albireo_sample takes from
// the caller's workspace lives here in a fixed array in the library's own device image.  Every GPU
// that loads the library holds it (4 MiB) until the process exits.

static __device__ __align__(256) uint32_t g_fixed_counts[ALBIREO_FIXED_MAX_HISTORY];

namespace {
constexpr int FIXED_MAX_DEVICES = 64;
struct FixedDeviceState {
    bool ready;
    uint32_t *counts;     // device address of g_fixed_counts on that device
    size_t max_smem;
    int num_sms;
};
FixedDeviceState g_fixed_dev[FIXED_MAX_DEVICES];
std::mutex g_fixed_mutex;
thread_local char g_fixed_err[256] = "";

int fixed_fail(int code, const char *fmt, const char *detail) {
    snprintf(g_fixed_err, sizeof g_fixed_err, fmt, detail ? detail : "");
    return code;
}

// Once per device, with that device current: the device address of the scratch array (its name
// in host code is only a stand-in, never something a kernel may be given) and the kernels'
// shared-memory opt-in.
int fixed_setup(int dev, FixedDeviceState **out) {
    if (dev < 0 || dev >= FIXED_MAX_DEVICES) return fixed_fail(ALBIREO_EUNSUPPORTED, "device index beyond what the fixed-scratch entry supports%s", "");
    std::lock_guard<std::mutex> lock(g_fixed_mutex);
    FixedDeviceState &d = g_fixed_dev[dev];
    if (!d.ready) {
        void *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_fixed_counts);
        if (e != cudaSuccess || !ptr) { cudaGetLastError(); return fixed_fail(ALBIREO_ECUDA, "cudaGetSymbolAddress failed: %s", cudaGetErrorString(e)); }
        const size_t smem = enable_large_smem(dev, &e);
        if (e != cudaSuccess) { cudaGetLastError(); return fixed_fail(ALBIREO_ECUDA, "kernel set-up failed: %s", cudaGetErrorString(e)); }
        d.num_sms = 0;
        if (cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) { cudaGetLastError(); d.num_sms = 0; }
        d.counts = (uint32_t *)ptr; d.max_smem = smem; d.ready = true;
    }
    *out = &d;
    return ALBIREO_OK;
}
}  // namespace

extern "C" int albireo_sample_fixed_scratch(const void *logits, int32_t B, int32_t V, int32_t dtype,
                                            const float *temperature, const int32_t *top_k, const float *top_p,
                                            const float *min_p, const float *repetition_penalty,
                                            const float *presence_penalty, const float *frequency_penalty,
                                            const int32_t *history_ids, const int32_t *history_offsets,
                                            int64_t history_total, const uint64_t *seeds, uint64_t step,
                                            int32_t *out_tokens, float *out_logprobs, void *stream,
                                            const albireo_sample_ext_t *ext) {
    g_fixed_err[0] = 0;
    if (B == 0) return ALBIREO_OK;
    if (B < 0) return fixed_fail(ALBIREO_EINVAL, "B is negative%s", "");
    if (V < 1) return fixed_fail(ALBIREO_EINVAL, "V is not positive%s", "");
    if (V > ALBIREO_MAX_VOCAB) return fixed_fail(ALBIREO_EUNSUPPORTED, "V exceeds ALBIREO_MAX_VOCAB%s", "");
    if (dtype != ALBIREO_F32 && dtype != ALBIREO_BF16 && dtype != ALBIREO_F16) return fixed_fail(ALBIREO_EINVAL, "unknown dtype%s", "");
    if (!logits || !out_tokens || !out_logprobs) return fixed_fail(ALBIREO_EINVAL, "NULL logits or output%s", "");
    if ((history_ids == nullptr) != (history_offsets == nullptr)) return fixed_fail(ALBIREO_EINVAL, "history_ids and history_offsets must both be given%s", "");
    if (history_total < 0) return fixed_fail(ALBIREO_EINVAL, "history_total is negative%s", "");
    if (history_total > (int64_t)ALBIREO_FIXED_MAX_HISTORY)
        return fixed_fail(ALBIREO_EUNSUPPORTED, "history_total exceeds ALBIREO_FIXED_MAX_HISTORY (the fixed scratch array); use albireo_sample with a workspace%s", "");
    const size_t esize = dtype == ALBIREO_F32 ? 4 : 2;
    if ((uintptr_t)logits % esize) return fixed_fail(ALBIREO_EINVAL, "logits not element-aligned%s", "");

    SampleArgs a;
    memset(&a, 0, sizeof a);
    a.logits = logits; a.B = B; a.V = V; a.row_stride = V; a.nseg = 1; a.Vs = V; a.vps = 0x7FFFFFFF; a.elem_size = (int32_t)esize;
    a.temperature = temperature; a.top_k = top_k; a.top_p = top_p; a.min_p = min_p;
    a.rep = repetition_penalty; a.pres = presence_penalty; a.freq = frequency_penalty;
    a.hist_ids = history_ids; a.hist_off = history_offsets;
    a.seeds = seeds; a.step = step;
    a.out_tokens = out_tokens; a.out_logprobs = out_logprobs;
    if (ext) {
        const char *why = nullptr;
        const int rc = apply_ext(a, ext, B, V, &why);
        if (rc != ALBIREO_OK) return fixed_fail(rc, "%s", why);
    }
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return fixed_fail(ALBIREO_ECUDA, "cudaGetDevice failed%s", ""); }
    FixedDeviceState *d = nullptr;
    const int rc = fixed_setup(dev, &d);
    if (rc != ALBIREO_OK) return rc;
    a.ws_counts = d->counts;                       // a device address, from cudaGetSymbolAddress
    a.ws_counts_cap = ALBIREO_FIXED_MAX_HISTORY;

    a.nstages = ring_stages_for(V, history_ids != nullptr, B <= d->num_sms);
    size_t smem = smem_bytes_for(V, history_ids != nullptr, a.nstages);
    while (smem > d->max_smem && a.nstages > 2) smem = smem_bytes_for(V, history_ids != nullptr, --a.nstages);
    if (smem > d->max_smem) return fixed_fail(ALBIREO_EUNSUPPORTED, "vocabulary too large for the on-chip tables%s", "");
    cudaStream_t st = (cudaStream_t)stream;
    launch_sample_kernel(dtype, B, smem, st, a);
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fixed_fail(ALBIREO_ECUDA, "kernel launch failed: %s", cudaGetErrorString(e));
    return ALBIREO_OK;
}

extern "C" const char *albireo_sample_fixed_scratch_error(void) { return g_fixed_err; }
