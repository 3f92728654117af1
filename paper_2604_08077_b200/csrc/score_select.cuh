// K3: cube scoring (Eq. 1) and nucleus selection (Eq. 2).
//
// Selection must reproduce an fp64 evaluation of Eqs. 1-2 bit for bit (only rows whose
// cumulative-probability margin is below 1e-6 may differ), so the scores are computed in fp64:
// Q is exact bf16, the mean keys are fp32, every product is exact in fp64 and the fp64 tensor
// op (mma.m8n8k4.f64) accumulates them.  The scores of a chunk of query tiles are staged in an
// L2-sized scratch buffer and consumed by the selection kernel of the same chunk; the full
// score matrix is never materialised.
//
//   score_kernel   CTA = 128 query rows (one tile) x 64 cubes, 8 warps of 32 x 32.
//   select_kernel  one warp per query row: softmax statistics, then a value-space quickselect
//                  for the nucleus boundary (no sort), then one ballot per 32 cubes emits the
//                  row's bitmap words.
#pragma once
#include "common.cuh"

namespace adaspark {

constexpr int kScoreCols = 64;  // cubes per score CTA
constexpr int kScoreKC = 16;    // head-dim chunk staged per iteration
constexpr int kScorePitch = 20; // doubles per smem row: 20 = 4 mod 16 keeps 64-bit fragment loads conflict-free

// logits[(gt - gt0) * 128 + r][j] = scale * <q_row, kbar_j>, for j < candidates of the tile.
template <int D>
__global__ void __launch_bounds__(256) score_kernel(Geom g, int gt0,
                                                    const __nv_bfloat16* __restrict__ q,
                                                    const float* __restrict__ cube_keys,
                                                    double* __restrict__ logits) {
    __shared__ double Qs[kTileRows][kScorePitch];
    __shared__ double Ks[kScoreCols][kScorePitch];

    const int gt = gt0 + blockIdx.x;
    int tile, bh, h, b;
    g.div_n_tiles.divmod(gt, bh, tile);
    g.div_Hq.divmod(bh, b, h);
    const int gk = h / g.G;
    const int col0 = blockIdx.y * kScoreCols;
    // candidates of the last valid row bound the columns this tile needs
    int last_pos = min(tile * kTileRows + kTileRows, g.S) - 1;
    if (col0 >= n_candidates(g, last_pos)) return;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wr = warp >> 1, wc = warp & 1;

    // each thread stages 8 query elements (row = tid/2) and 4 key elements (cube = tid/4)
    const int qrow = tid >> 1, qhalf = tid & 1;
    const int qpos = tile * kTileRows + qrow;
    const __nv_bfloat16* qsrc = nullptr;
    if (qpos < g.S) qsrc = q + ((size_t)(b * g.S + pos_to_raster(g, qpos)) * g.Hq + h) * D;
    const int kcube = tid >> 2, kq = tid & 3;
    const float* ksrc = nullptr;
    if (col0 + kcube < g.N) ksrc = cube_keys + ((size_t)(b * g.Hkv + gk) * g.N + col0 + kcube) * D;

    double acc[4][4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;

    for (int k0 = 0; k0 < D; k0 += kScoreKC) {
        uint4 qv = make_uint4(0, 0, 0, 0);
        if (qsrc) qv = *reinterpret_cast<const uint4*>(qsrc + k0 + qhalf * 8);
        float4 kv = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ksrc) kv = *reinterpret_cast<const float4*>(ksrc + k0 + kq * 4);
        __syncthreads();  // previous chunk fully consumed
        const __nv_bfloat162* q2 = reinterpret_cast<const __nv_bfloat162*>(&qv);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f = __bfloat1622float2(q2[i]);
            Qs[qrow][qhalf * 8 + 2 * i] = (double)f.x;
            Qs[qrow][qhalf * 8 + 2 * i + 1] = (double)f.y;
        }
        Ks[kcube][kq * 4 + 0] = (double)kv.x;
        Ks[kcube][kq * 4 + 1] = (double)kv.y;
        Ks[kcube][kq * 4 + 2] = (double)kv.z;
        Ks[kcube][kq * 4 + 3] = (double)kv.w;
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kScoreKC; kk += 4) {
            double a[4], bb[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = Qs[wr * 32 + i * 8 + (lane >> 2)][kk + (lane & 3)];
#pragma unroll
            for (int j = 0; j < 4; ++j) bb[j] = Ks[wc * 32 + j * 8 + (lane >> 2)][kk + (lane & 3)];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) mma_f64_884(acc[i][j], a[i], bb[j]);
        }
    }

    double* base = logits + (size_t)(blockIdx.x) * kTileRows * g.N_ld;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int r = wr * 32 + i * 8 + (lane >> 2);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int c = col0 + wc * 32 + j * 8 + 2 * (lane & 3);
            double2 o = make_double2(acc[i][j][0] * g.scale_d, acc[i][j][1] * g.scale_d);
            *reinterpret_cast<double2*>(base + (size_t)r * g.N_ld + c) = o;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// Nucleus boundary of one row, executed by one full warp.
//
// Cubes are ordered by (probability descending, index ascending); the nucleus is the shortest
// prefix of that order whose mass reaches the target.  Each candidate j is represented by one
// 64-bit ORDER KEY: the bit pattern of e_j = exp(s_j - max) >= 0 (non-negative doubles order like
// their bit patterns) with its 13 lowest mantissa bits replaced by (4096 - j).  A larger key comes
// earlier in the order; equal probabilities are ordered by lower index.  Replacing the low
// mantissa bits changes a value by less than 2^-39 relative, far below the 1e-6 tie margin that
// bounds which rows may legitimately differ from an exact evaluation.  Keys are never zero.
//
// The search narrows an open interval (hi_key < key < lo_key) around the boundary: each pass picks
// one interval element as pivot, sums the interval's mass above the pivot (warp reduction) and
// keeps the side that holds the crossing.  Returns the boundary key: cube j is selected iff
// key_j >= boundary (0 selects everything).
// ---------------------------------------------------------------------------------------------
constexpr unsigned long long kIdxMask = 0x1FFFull;

__device__ __forceinline__ unsigned long long order_key(double e, int j) {
    return ((unsigned long long)__double_as_longlong(e) & ~kIdxMask) | (unsigned long long)(4096 - j);
}
__device__ __forceinline__ double key_mass(unsigned long long key) {
    return __longlong_as_double((long long)(key & ~kIdxMask));
}

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

__device__ unsigned long long nucleus_boundary(const unsigned long long* keys, int n, double target, int lane) {
    unsigned long long lo = ~0ull, hi = 0ull;   // interval: hi < key < lo
    double base = 0.0;                          // mass of every key >= lo
    unsigned long long cand = lane < n ? keys[lane] : 0ull;   // each lane offers one interval element
    for (int iter = 0; iter < n + 2; ++iter) {
        const uint32_t have = __ballot_sync(0xffffffffu, cand != 0ull);
        if (have == 0u) break;
        // pivot: the offer of one offering lane, rotating the starting lane every pass (offers are
        // in index order, i.e. unordered in value)
        const int rot = (iter * 11) & 31;
        const int src = (__ffs(__funnelshift_r(have, have, rot)) - 1 + rot) & 31;
        const unsigned long long pv = __shfl_sync(0xffffffffu, cand, src);
        double mass_above = 0.0;
        unsigned long long cand_above = 0ull, cand_below = 0ull;
        for (int j = lane; j < n; j += 32) {
            const unsigned long long kj = keys[j];
            if (kj >= lo || kj <= hi) continue;
            if (kj > pv) {
                mass_above += key_mass(kj);
                if (cand_above == 0ull) cand_above = kj;
            } else if (kj < pv) {
                if (cand_below == 0ull) cand_below = kj;
            }
        }
        mass_above = warp_sum(mass_above);
        const double pv_mass = key_mass(pv);
        if (base + mass_above >= target) {              // crossing strictly above the pivot
            hi = pv;
            cand = cand_above;
        } else if (base + mass_above + pv_mass >= target) {
            return pv;                                   // the pivot is the crossing element
        } else {
            base += mass_above + pv_mass;
            lo = pv;
            cand = cand_below;
        }
    }
    // Interval exhausted without reaching the target (rounding of partial sums): keep all above hi.
    return hi == 0ull ? 0ull : lo;
}

// ---------------------------------------------------------------------------------------------
// Radix selection of the nucleus boundary on integer order keys (one warp per row).
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
// memory, lane b then sums bucket b over the 32 columns, and a warp scan finds the bucket in which
// the cumulative mass crosses T.  As soon as at most 32 keys remain in the interval they are spread
// over the lanes and the crossing key is found directly (mass of all keys >= mine, all pairs).
// ---------------------------------------------------------------------------------------------
constexpr int kSelHistPitch = 33;                       // u64 per histogram row: padded, conflict-free column sums
constexpr int kSelHistWords = 32 * kSelHistPitch;       // u64 per warp
constexpr int kSelCandCap = 256;                        // compacted interval members kept per warp
constexpr int kSelWarpScratch = kSelHistWords + kSelCandCap;   // u64 per warp besides the keys

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
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
    if (b & 1) { lo = base; hi = base + half - 1ull; }          // second = 0
    else       { lo = base + half; hi = base + half + half - 1ull; }   // second = 1
}
__device__ __forceinline__ int octave_bucket_of(int top, unsigned long long key) {
    const int lead = 63 - __clzll((long long)key);
    const int second = lead > 0 ? (int)((key >> (lead - 1)) & 1ull) : 0;
    const int b = 2 * (top - lead) + 1 - second;
    return b > 31 ? 31 : (b < 0 ? 0 : b);
}

// Sums the 32 private columns of every bucket (lane b owns bucket b), scans the buckets from the
// top of the order and returns the bucket in which base + cumulative mass first reaches `target`;
// `base` is advanced by the mass of the buckets before it.
__device__ __forceinline__ int crossing_bucket(const unsigned long long* hist, int lane, unsigned long long target,
                                               unsigned long long& base) {
    unsigned long long mine = 0ull;
    const unsigned long long* row = hist + lane * kSelHistPitch;
#pragma unroll
    for (int l = 0; l < 32; ++l) mine += row[l];
    unsigned long long incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    const uint32_t reach = __ballot_sync(0xffffffffu, base + incl >= target);
    const int c = reach ? __ffs(reach) - 1 : 31;          // exact integer sums: some bucket always reaches
    const unsigned long long before = __shfl_sync(0xffffffffu, incl - mine, c);
    base += before;
    return c;
}

__device__ __forceinline__ void zero_hist(unsigned long long* hist, int lane) {
    uint4* h4 = reinterpret_cast<uint4*>(hist);
    for (int i = lane; i < kSelHistWords / 2; i += 32) h4[i] = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();
}

// Finds the boundary key of one row.  On entry keys[0..n) hold the order keys, `hist` holds the
// first-level histogram (half-octave buckets with top = 63) and `target` = T.  `cand` is scratch.
__device__ unsigned long long radix_boundary(const unsigned long long* keys, int n, unsigned long long target,
                                             unsigned long long* hist, unsigned long long* cand, int lane) {
    unsigned long long base = 0ull, lo, hi;
    int top = 63;
    int c = crossing_bucket(hist, lane, target, base);
    octave_bucket_range(top, c, lo, hi);
    bool octave_split = (c == 31);          // the crossing lies in the overflow bucket: split it again
    int shift = c == 31 ? 0 : (top - (c >> 1)) - 6;   // next 5 bits below (lead, second)
    if (shift < 0) shift = 0;
    if (c == 31) top -= 15;
    const unsigned long long* src = keys;
    int len = n;
    for (int level = 0; level < 24; ++level) {
        // gather the interval members (compacted into cand while they fit)
        int count = 0;
        for (int i0 = 0; i0 < len; i0 += 32) {
            const int i = i0 + lane;
            const unsigned long long k = i < len ? src[i] : 0ull;
            const bool in = k >= lo && k <= hi;
            const uint32_t ball = __ballot_sync(0xffffffffu, in);
            const int pos = count + __popc(ball & ((1u << lane) - 1u));
            if (in && pos < kSelCandCap) cand[pos] = k;
            count += __popc(ball);
        }
        __syncwarp();
        if (count <= 32) {
            // one key per lane: the crossing key is the largest key whose "mass of all keys >= it"
            // reaches the target
            const unsigned long long mine = lane < count ? cand[lane] : 0ull;
            unsigned long long acc = 0ull;
#pragma unroll 8
            for (int l = 0; l < 32; ++l) {
                const unsigned long long other = __shfl_sync(0xffffffffu, mine, l);
                if (other >= mine) acc += other >> 13;
            }
            const bool reach = lane < count && base + acc >= target;
            uint32_t hi32 = reach ? (uint32_t)(mine >> 32) : 0u;
            const uint32_t best_hi = __reduce_max_sync(0xffffffffu, hi32);
            uint32_t lo32 = (reach && hi32 == best_hi) ? (uint32_t)mine : 0u;
            const uint32_t best_lo = __reduce_max_sync(0xffffffffu, lo32);
            return ((unsigned long long)best_hi << 32) | best_lo;
        }
        if (count <= kSelCandCap) { src = cand; len = count; }
        // next level over the interval members
        zero_hist(hist, lane);
        for (int i = lane; i < len; i += 32) {
            const unsigned long long k = src[i];
            if (k >= lo && k <= hi) {
                const int b = octave_split ? octave_bucket_of(top, k) : 31 - (int)((k >> shift) & 31ull);
                hist[b * kSelHistPitch + lane] += k >> 13;
            }
        }
        __syncwarp();
        c = crossing_bucket(hist, lane, target, base);
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
    return lo;   // not reached: keys are distinct, so the interval shrinks to one key well before
}

// Builds the order keys of one row from its scaled scores s[0..n) (fp64), fills the first-level
// histogram and returns the boundary key: cube j is selected iff keys[j] >= boundary.
// keys: n entries; scratch: kSelWarpScratch entries.  n >= 1, p < 1.
__device__ unsigned long long nucleus_boundary_radix(const double* __restrict__ s, int n, double top_p,
                                                     unsigned long long* keys, unsigned long long* scratch, int lane) {
    unsigned long long* hist = scratch;
    unsigned long long* cand = scratch + kSelHistWords;
    zero_hist(hist, lane);
    double* sd = reinterpret_cast<double*>(keys);
    double mx = -INFINITY;
    for (int j = lane; j < n; j += 32) {
        const double v = s[j];
        sd[j] = v;
        mx = fmax(mx, v);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    unsigned long long z = 0ull;
    for (int j = lane; j < n; j += 32) {
        const double e = exp(sd[j] - mx);
        const double r = fma(e, 0x1p50, 0x1p52);                       // integer part of e * 2^50, rounded to nearest
        const unsigned long long m = (unsigned long long)__double_as_longlong(r) & 0xFFFFFFFFFFFFFull;
        const int top_bits = __double2hiint(r - 0x1p52) >> 19;        // (exponent << 1) | top mantissa bit of (double)m
        int b = 2147 - top_bits;                                      // m = 2^50 -> 1, each half octave below -> +1
        b = b > 31 ? 31 : b;
        keys[j] = (m << 13) | (unsigned long long)(4096 - j);
        hist[b * kSelHistPitch + lane] += m;
        z += m;
    }
    z = warp_sum_u64(z);
    __syncwarp();
    const unsigned long long target = (unsigned long long)ceil((double)z * top_p);
    return radix_boundary(keys, n, target, hist, cand, lane);
}

// One warp per query row of the chunk.  Writes the per-tile mask matrix (always) and the
// optional raster-ordered bitmap / count outputs.
// dynamic smem: per warp N_ld keys + kSelWarpScratch words of 8 bytes.
constexpr int kSelectWarps = 4;
__host__ __device__ inline size_t select_smem_bytes(int N_ld) {
    return (size_t)kSelectWarps * ((size_t)N_ld + kSelWarpScratch) * 8;
}

__global__ void __launch_bounds__(kSelectWarps * 32) select_kernel(Geom g, int gt0, int n_gt,
                                                     const double* __restrict__ logits,
                                                     uint32_t* __restrict__ tile_mask,
                                                     uint32_t* __restrict__ sel_bitmap,
                                                     int32_t* __restrict__ sel_count) {
    extern __shared__ __align__(16) unsigned long long sel_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row_id = blockIdx.x * kSelectWarps + warp;        // row within the chunk
    if (row_id >= n_gt * kTileRows) return;
    const int gt = gt0 + row_id / kTileRows, r = row_id % kTileRows;
    int tile, bh, h, b;
    g.div_n_tiles.divmod(gt, bh, tile);
    g.div_Hq.divmod(bh, b, h);
    const int pos = tile * kTileRows + r;
    unsigned long long* scratch = sel_smem + (size_t)warp * kSelWarpScratch;
    unsigned long long* keys = sel_smem + (size_t)kSelectWarps * kSelWarpScratch + (size_t)warp * g.N_ld;
    const double* s = logits + (size_t)row_id * g.N_ld;

    const int n = pos < g.S ? n_candidates(g, pos) : 0;
    unsigned long long bd = 0ull;                    // default: every candidate is selected
    const bool all = !(g.top_p < 1.0);
    if (n > 0 && !all) bd = nucleus_boundary_radix(s, n, g.top_p, keys, scratch, lane);

    const bool extra = (sel_bitmap != nullptr || sel_count != nullptr) && pos < g.S;
    const int raster = extra ? pos_to_raster(g, pos) : 0;
    int count = 0;
    for (int w = 0; w < g.n_words; ++w) {
        int j = w * 32 + lane;
        bool on = j < n && (all || keys[j] >= bd);
        uint32_t word = __ballot_sync(0xffffffffu, on);
        count += __popc(word);
        if (lane == 0) {
            tile_mask[mask_index(g, b, h, tile, w, r)] = word;
            if (sel_bitmap && extra)
                sel_bitmap[((size_t)(b * g.Hq + h) * g.S + raster) * g.n_words + w] = word;
        }
    }
    if (sel_count && lane == 0 && extra) sel_count[(size_t)(b * g.Hq + h) * g.S + raster] = count;
}

}  // namespace adaspark
