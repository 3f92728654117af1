// Nucleus (Top-p) boundary of Eq. 2 by radix selection on exact integer order keys.
//
// A warp serves 32/G query rows at once, G lanes per row (G = 8, 16 or 32): short candidate lists
// share the fixed per-warp work (histogram column sums, scans, the final all-pairs step) between
// several rows.  Everything below is written for a "group" = the G lanes of one row; all 32 lanes
// always take part in the warp collectives, a group without work simply carries n = 0.
//
// Every candidate j gets the fixed-point mass m_j = round(exp(s_j - max) * 2^50) (an integer in
// [0, 2^50]; the row maximum has exactly 2^50) and the 64-bit ORDER KEY
//     key_j = (m_j << 13) | (4096 - j)          (never zero, all keys of a row distinct).
// A larger key comes earlier in the order (probability descending, equal masses by lower cube
// index).  With Z = sum m_j the nucleus is the shortest prefix of that order whose mass reaches
// T = ceil(p * Z); all sums are exact integer sums, so the result does not depend on the order of
// accumulation.  Quantising a probability to 2^-50 of the row maximum moves no cumulative sum by
// more than 4096 * 2^-51 of Z, ten orders of magnitude below the 1e-6 margin inside which a row
// may legitimately differ from an fp64 evaluation of Eqs. 1-2.
//
// The boundary key (smallest selected key) is found by narrowing a key interval [lo, hi] that
// holds the crossing element, 32 buckets at a time:
//   first level   half-octave buckets of the key (position of the leading bit + the bit below it),
//                 filled while the keys are produced; an overflow bucket catches everything more
//                 than 15 octaves below the current top and is re-split if the crossing lies there;
//   next levels   the next 5 key bits below the bits already fixed.
// Per level each lane adds the masses of its keys to a private histogram column in shared
// memory, the lanes of the group then sum the 32 buckets over the group's columns, and a scan finds
// the bucket in which the cumulative mass crosses T.  As soon as at most 32 keys remain in the
// interval they are spread over the group's lanes and the crossing key is found directly (mass of
// all keys >= mine, all pairs).
#pragma once
#include "common.cuh"

namespace adaspark {

// exp(x) for x <= 0 with a relative error below 1e-12 (argument reduction by ln 2, degree-10 Taylor
// polynomial on |r| <= 0.347, exponent added as an integer): less than half the instructions of the
// library routine.  The selection needs probabilities only far more accurately than the 1e-6 margin
// inside which a row may differ from an fp64 evaluation, not to the last bit.  exp(-inf) and
// anything below 2^-1020 return 0.
__device__ __forceinline__ double exp_nonpositive(double x) {
    const double t = fma(x, 1.4426950408889634, 6755399441055744.0);   // rint(x * log2 e) in the low word
    const int k = __double2loint(t);
    const double kd = t - 6755399441055744.0;
    double r = fma(kd, -6.93147180369123816490e-01, x);
    r = fma(kd, -1.90821492927058770002e-10, r);
    double p = 2.7557319223985893e-07;                                  // 1/10!
    p = fma(p, r, 2.7557319223985888e-06);
    p = fma(p, r, 2.4801587301587302e-05);
    p = fma(p, r, 1.9841269841269841e-04);
    p = fma(p, r, 1.3888888888888889e-03);
    p = fma(p, r, 8.3333333333333332e-03);
    p = fma(p, r, 4.1666666666666664e-02);
    p = fma(p, r, 1.6666666666666666e-01);
    p = fma(p, r, 0.5);
    p = fma(p, r, 1.0);
    p = fma(p, r, 1.0);
    const double scaled = __hiloint2double(__double2hiint(p) + (int)((unsigned)k << 20), __double2loint(p));
    return (x > -707.0) ? scaled : 0.0;
}

constexpr int kSelHistWords = 32 * 32;   // u64 per warp: [bucket][lane column], columns rotated per bucket

template <int G>
struct SelGeom {
    static_assert(G == 8 || G == 16 || G == 32, "lanes per row");
    static constexpr int kRows = 32 / G;                               // rows per warp
    static constexpr int kOwn = 32 / G;                                // buckets (and final-step slots) per lane
    static constexpr int kOwnShift = G == 32 ? 0 : (G == 16 ? 1 : 2);  // log2(kOwn)
};

// Column `col` of bucket b lives at a rotated position so that both the private updates and the
// column sums (lane of the group that owns bucket b reads the group's columns) spread over the banks.
template <int G>
__device__ __forceinline__ int hist_index(int b, int col) {
    return b * 32 + ((col + (b >> SelGeom<G>::kOwnShift)) & 31);
}

__device__ __forceinline__ void zero_hist(unsigned long long* hist, int lane) {
    uint4* h4 = reinterpret_cast<uint4*>(hist);
#pragma unroll
    for (int i = 0; i < kSelHistWords / 2 / 32; ++i) h4[lane + 32 * i] = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();
}

// Key interval of bucket b of a half-octave split whose first octave has its leading bit at `top`:
// bucket 2*(top-lead) + 1 - second, clamped to 31 (second = the bit below the leading bit).
__device__ __forceinline__ void octave_bucket_range(int top, int b, unsigned long long& lo, unsigned long long& hi) {
    if (b >= 31) {                      // everything below bucket 30 = (lead = top-15, second = 1)
        lo = 1ull;
        hi = (1ull << (top - 15)) + (1ull << (top - 16)) - 1ull;
        return;
    }
    const int lead = top - (b >> 1);
    const unsigned long long base = 1ull << lead, half = 1ull << (lead - 1);
    if (b & 1) { lo = base; hi = base + half - 1ull; }                 // second = 0
    else       { lo = base + half; hi = base + half + half - 1ull; }   // second = 1
}
__device__ __forceinline__ int octave_bucket_of(int top, unsigned long long key) {
    const int lead = 63 - __clzll((long long)key);
    const int second = lead > 0 ? (int)((key >> (lead - 1)) & 1ull) : 0;
    const int b = 2 * (top - lead) + 1 - second;
    return b > 31 ? 31 : (b < 0 ? 0 : b);
}

// Column sums of the group's histogram, scan over the 32 buckets from the top of the order, and
// the first bucket in which base + cumulative mass reaches `target`.  `base` advances by the mass
// of the buckets before it.  (Exact integer sums: some bucket always reaches the target.)
template <int G>
__device__ __forceinline__ int crossing_bucket(const unsigned long long* hist, int lane, unsigned long long target,
                                               unsigned long long& base) {
    constexpr int kOwn = SelGeom<G>::kOwn;
    const int gl = lane & (G - 1), gbase = lane & ~(G - 1);
    unsigned long long pre[kOwn];       // inclusive prefix over this lane's buckets gl*kOwn .. +kOwn-1
    unsigned long long run = 0ull;
#pragma unroll
    for (int k = 0; k < kOwn; ++k) {
        const unsigned long long* row = hist + (gl * kOwn + k) * 32;
        unsigned long long sum = 0ull;
#pragma unroll
        for (int l = 0; l < G; ++l) sum += row[(gbase + l + gl) & 31];
        run += sum;
        pre[k] = run;
    }
    unsigned long long incl = run;      // inclusive scan of the lane totals inside the group
#pragma unroll
    for (int o = 1; o < G; o <<= 1) {
        const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
        if (gl >= o) incl += t;
    }
    const unsigned long long excl = incl - run;
    int kfirst = kOwn;
#pragma unroll
    for (int k = kOwn - 1; k >= 0; --k)
        if (base + excl + pre[k] >= target) kfirst = k;
    const uint32_t ball = __ballot_sync(0xffffffffu, kfirst < kOwn);
    const uint32_t mine = G == 32 ? ball : ((ball >> gbase) & ((1u << G) - 1u));
    const int f = mine ? __ffs(mine) - 1 : G - 1;
    const int kf = __shfl_sync(0xffffffffu, kfirst < kOwn ? kfirst : kOwn - 1, gbase + f);
    unsigned long long before = excl;
#pragma unroll
    for (int k = 1; k < kOwn; ++k)
        if (kf >= k) before = excl + pre[k - 1];
    before = __shfl_sync(0xffffffffu, before, gbase + f);
    base += before;
    return f * kOwn + kf;
}

template <int G>
__device__ __forceinline__ unsigned long long group_sum_u64(unsigned long long x) {
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Boundary key of each group's row.  On entry keys[0..n) of the group hold its order keys and the
// group's columns of `hist` hold the first-level histogram (half-octave buckets, top = 63);
// `target` = T.  `cand` is the group's scratch list of `cand_cap` entries.  A group with n = 0
// takes part in the collectives and returns 0.  by_count: every key weighs 1 instead of its mass (the
// histogram then counts keys and `target` is a rank: the Top-K rule).
template <int G>
__device__ unsigned long long radix_boundary(const unsigned long long* keys, int n, unsigned long long target,
                                             unsigned long long* hist, unsigned long long* cand, int cand_cap,
                                             int lane, bool by_count) {
    constexpr int kOwn = SelGeom<G>::kOwn;
    const int gl = lane & (G - 1), gbase = lane & ~(G - 1);
    const uint32_t gmask = G == 32 ? 0xffffffffu : (((1u << G) - 1u) << gbase);
    unsigned long long base = 0ull, lo, hi;
    int top = 63;
    int c = crossing_bucket<G>(hist, lane, target, base);
    octave_bucket_range(top, c, lo, hi);
    bool octave_split = (c == 31);          // the crossing lies in the overflow bucket: split it again
    int shift = c == 31 ? 0 : (top - (c >> 1)) - 6;   // next 5 bits below (lead, second)
    if (shift < 0) shift = 0;
    if (c == 31) top -= 15;
    const unsigned long long* src = keys;
    int len = n;
    int count = 0;
    bool done = (n == 0);
    for (int level = 0; level < 24; ++level) {
        // ---- members of the interval, compacted into cand while they fit
        const int len_max = __reduce_max_sync(0xffffffffu, done ? 0 : len);
        int cnt = 0;
        for (int i0 = 0; i0 < len_max; i0 += G) {
            const int i = i0 + gl;
            const unsigned long long k = (!done && i < len) ? src[i] : 0ull;
            const bool in = k >= lo && k <= hi && k != 0ull;
            const uint32_t ball = __ballot_sync(0xffffffffu, in) & gmask;
            const int pos = cnt + __popc(ball & ((1u << lane) - 1u));
            if (in && pos < cand_cap) cand[pos] = k;
            cnt += __popc(ball);
        }
        __syncwarp();
        if (!done) {
            count = cnt;
            if (count <= 32) done = true;
            else if (count <= cand_cap) { src = cand; len = count; }
        }
        if (__all_sync(0xffffffffu, done)) break;
        // ---- next level over the interval members of the groups that are not done
        zero_hist(hist, lane);
        if (!done) {
            for (int i = gl; i < len; i += G) {
                const unsigned long long k = src[i];
                if (k >= lo && k <= hi) {
                    const int b = octave_split ? octave_bucket_of(top, k) : 31 - (int)((k >> shift) & 31ull);
                    hist[hist_index<G>(b, lane)] += by_count ? 1ull : (k >> 13);
                }
            }
        }
        __syncwarp();
        unsigned long long nbase = base;
        c = crossing_bucket<G>(hist, lane, target, nbase);
        if (!done) {
            base = nbase;
            if (octave_split) {
                octave_bucket_range(top, c, lo, hi);
                if (c == 31) { top = top > 33 ? top - 15 : 18; }   // below 2^3 only zero-mass keys remain
                else { octave_split = false; shift = (top - (c >> 1)) - 6; }
            } else {
                const unsigned long long prefix = lo & ~((32ull << shift) - 1ull);
                lo = prefix | ((unsigned long long)(31 - c) << shift);
                hi = lo | ((1ull << shift) - 1ull);
                shift -= 5;
            }
            if (shift < 0) shift = 0;
        }
    }
    // ---- at most 32 keys per group: slot sl of lane gl holds cand[sl*G + gl].  The crossing key is
    // the largest key whose "mass of all keys >= it" reaches the target.
    unsigned long long mine[kOwn], acc[kOwn];
#pragma unroll
    for (int sl = 0; sl < kOwn; ++sl) {
        const int i = sl * G + gl;
        mine[sl] = (i < count && count <= 32) ? cand[i] : 0ull;
        acc[sl] = 0ull;
    }
    // every candidate of the group in turn, read from the list in shared memory (a broadcast load);
    // the loop runs to the longest list among the groups of the warp
    const int cmax = __reduce_max_sync(0xffffffffu, count <= 32 ? count : 0);
    for (int e = 0; e < cmax; ++e) {
        const unsigned long long other = e < count ? cand[e] : 0ull;
        const unsigned long long om = by_count ? (other != 0ull ? 1ull : 0ull) : (other >> 13);
#pragma unroll
        for (int sl = 0; sl < kOwn; ++sl)
            if (other >= mine[sl]) acc[sl] += om;
    }
    unsigned long long best = 0ull;
#pragma unroll
    for (int sl = 0; sl < kOwn; ++sl)
        if (mine[sl] != 0ull && base + acc[sl] >= target && mine[sl] > best) best = mine[sl];
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) {
        const unsigned long long t = __shfl_xor_sync(0xffffffffu, best, o);
        best = t > best ? t : best;
    }
    return best;
}

// Builds the order keys of the group's row from its scaled scores s[0..n) (fp64), fills the
// first-level histogram and returns the boundary key: cube j is selected iff keys[j] >= boundary.
// A group with n = 0 (no candidates, or nothing to search) returns 0.  Requires p < 1 or top_k > 0
// (top_k > 0 selects the min(top_k, n) first keys of the order instead of the nucleus).
// hist: kSelHistWords entries shared by the warp (zeroed here); keys / cand: the group's own.
// keys may be the score row itself (kInPlace: every score is replaced by its key, e.g. a row of the
// L2-resident score buffer) or separate storage (shared memory for short rows).
template <int G, bool kInPlace>
__device__ unsigned long long nucleus_boundary_radix(const double* s, int n, double top_p, int top_k,
                                                     unsigned long long* keys, unsigned long long* hist,
                                                     unsigned long long* cand, int cand_cap, int lane) {
    const int gl = lane & (G - 1);
    const bool by_count = top_k > 0;
    zero_hist(hist, lane);
    double* sd = reinterpret_cast<double*>(keys);
    double mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
    int j = gl;
    for (; j + 3 * G < n; j += 4 * G) {                 // four independent loads in flight per lane
        const double v0 = s[j], v1 = s[j + G], v2 = s[j + 2 * G], v3 = s[j + 3 * G];
        if (!kInPlace) { sd[j] = v0; sd[j + G] = v1; sd[j + 2 * G] = v2; sd[j + 3 * G] = v3; }
        mx0 = fmax(mx0, v0); mx1 = fmax(mx1, v1); mx2 = fmax(mx2, v2); mx3 = fmax(mx3, v3);
    }
    for (; j < n; j += G) {
        const double v = s[j];
        if (!kInPlace) sd[j] = v;
        mx0 = fmax(mx0, v);
    }
    double mx = fmax(fmax(mx0, mx1), fmax(mx2, mx3));
#pragma unroll
    for (int o = G / 2; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    unsigned long long z = 0ull;
    // mass, order key and first-level bucket of one candidate
    auto make_key = [&](double v, int jj, unsigned long long& m, int& b) -> unsigned long long {
        const double e = exp_nonpositive(v - mx);
        const double r = fma(e, 0x1p50, 0x1p52);                       // integer part of e * 2^50, rounded to nearest
        m = (unsigned long long)__double_as_longlong(r) & 0xFFFFFFFFFFFFFull;
        const int top_bits = __double2hiint(r - 0x1p52) >> 19;        // (exponent << 1) | top mantissa bit of (double)m
        b = 2147 - top_bits;                                          // m = 2^50 -> 1, each half octave below -> +1
        b = b > 31 ? 31 : (b < 0 ? 0 : b);                            // (non-finite scores must not index out of range)
        return (m << 13) | (unsigned long long)(4096 - jj);
    };
    j = gl;
    for (; j + 3 * G < n; j += 4 * G) {                 // four exponentials interleaved, then the four updates
        unsigned long long m[4], k[4];
        int b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) k[u] = make_key(sd[j + u * G], j + u * G, m[u], b[u]);
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            keys[j + u * G] = k[u];
            hist[hist_index<G>(b[u], lane)] += by_count ? 1ull : m[u];
            z += by_count ? 1ull : m[u];
        }
    }
    for (; j < n; j += G) {
        unsigned long long m;
        int b;
        keys[j] = make_key(sd[j], j, m, b);
        hist[hist_index<G>(b, lane)] += by_count ? 1ull : m;
        z += by_count ? 1ull : m;
    }
    z = group_sum_u64<G>(z);
    __syncwarp();
    // Top-p: mass target ceil(p * Z);  Top-K: the K-th key of the order (all of them if fewer exist)
    const unsigned long long target = by_count ? (z < (unsigned long long)top_k ? z : (unsigned long long)top_k)
                                               : (unsigned long long)ceil((double)z * top_p);
    return radix_boundary<G>(keys, n, target, hist, cand, cand_cap, lane, by_count);
}

}  // namespace adaspark
