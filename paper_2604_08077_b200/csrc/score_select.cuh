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
    const int tile = gt % g.n_tiles, bh = gt / g.n_tiles;
    const int h = bh % g.Hq, b = bh / g.Hq;
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

// One warp per query row of the chunk.  Writes the per-tile mask matrix (always) and the
// optional raster-ordered bitmap / count outputs.  dynamic smem: warps_per_cta * N_ld keys.
__global__ void __launch_bounds__(128) select_kernel(Geom g, int gt0, int n_gt,
                                                     const double* __restrict__ logits,
                                                     uint32_t* __restrict__ tile_mask,
                                                     uint32_t* __restrict__ sel_bitmap,
                                                     int32_t* __restrict__ sel_count) {
    extern __shared__ unsigned long long sel_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row_id = blockIdx.x * 4 + warp;        // row within the chunk
    if (row_id >= n_gt * kTileRows) return;
    const int gt = gt0 + row_id / kTileRows, r = row_id % kTileRows;
    const int tile = gt % g.n_tiles, bh = gt / g.n_tiles;
    const int h = bh % g.Hq, b = bh / g.Hq;
    const int pos = tile * kTileRows + r;
    unsigned long long* keys = sel_smem + (size_t)warp * g.N_ld;
    const double* s = logits + (size_t)row_id * g.N_ld;

    const int n = pos < g.S ? n_candidates(g, pos) : 0;
    unsigned long long bd = 0ull;                    // default: every candidate is selected
    if (n > 0 && g.top_p < 1.0) {
        double mx = -INFINITY;
        for (int j = lane; j < n; j += 32) mx = fmax(mx, s[j]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        double z = 0.0;
        for (int j = lane; j < n; j += 32) {
            double ej = exp(s[j] - mx);
            keys[j] = order_key(ej, j);
            z += ej;
        }
        z = warp_sum(z);
        __syncwarp();
        bd = nucleus_boundary(keys, n, g.top_p * z, lane);
    } else {
        for (int j = lane; j < n; j += 32) keys[j] = order_key(1.0, j);
        __syncwarp();
    }

    const int raster = pos < g.S ? pos_to_raster(g, pos) : 0;
    int count = 0;
    for (int w = 0; w < g.n_words; ++w) {
        int j = w * 32 + lane;
        bool on = j < n && keys[j] >= bd;
        uint32_t word = __ballot_sync(0xffffffffu, on);
        count += __popc(word);
        if (lane == 0) {
            tile_mask[mask_index(g, b, h, tile, w, r)] = word;
            if (sel_bitmap && pos < g.S)
                sel_bitmap[((size_t)(b * g.Hq + h) * g.S + raster) * g.n_words + w] = word;
        }
    }
    if (sel_count && lane == 0 && pos < g.S) sel_count[(size_t)(b * g.Hq + h) * g.S + raster] = count;
}

}  // namespace adaspark
