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
//   e[0..n)   unnormalised probabilities exp(s_j - max) as doubles in shared memory (all >= 0)
//   target    top_p * sum(e)
// Cubes are ordered by (e descending, index ascending); the nucleus is the shortest prefix of
// that order whose mass reaches target.  Returns the boundary element (key bits, index): cube j
// is selected iff it precedes or equals the boundary.  The search narrows an open interval
// (lo, hi) of the order around the boundary: each pass takes one pivot from the interval, sums
// the interval's mass that precedes the pivot, and keeps the side holding the crossing.
// Non-negative doubles order like their bit patterns, so all comparisons are on integers.
// ---------------------------------------------------------------------------------------------
struct OrderKey {
    unsigned long long key;
    int idx;
};
__device__ __forceinline__ bool precedes(unsigned long long ka, int ia, unsigned long long kb, int ib) {
    return ka > kb || (ka == kb && ia < ib);
}

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Sort 32 (key, idx) pairs, one per lane, into the selection order (bitonic network via shuffles).
__device__ __forceinline__ void warp_sort_order(unsigned long long& key, int& idx, int lane) {
#pragma unroll
    for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            unsigned long long ok = __shfl_xor_sync(0xffffffffu, key, j);
            int oi = __shfl_xor_sync(0xffffffffu, idx, j);
            bool up = ((lane & k) == 0);          // ascending segment (in selection order)
            bool lower = ((lane & j) == 0);       // this lane keeps the earlier element
            bool other_first = precedes(ok, oi, key, idx);
            bool take = (lower == up) ? other_first : !other_first;
            if (take) { key = ok; idx = oi; }
        }
    }
}

__device__ OrderKey nucleus_boundary(const double* e, int n, double target, int lane) {
    const unsigned long long* ek = reinterpret_cast<const unsigned long long*>(e);
    // open interval (lo, hi): lo precedes every element, hi follows every element
    unsigned long long lo_k = ~0ull, hi_k = 0ull;
    int lo_i = -1, hi_i = 0x7fffffff;
    double base = 0.0;  // mass of everything that precedes or equals lo
    // first pivot candidates: each lane offers its first element
    unsigned long long cand_k = 0ull;
    int cand_i = 0x7fffffff;
    if (lane < n) { cand_k = ek[lane]; cand_i = lane; }
    int n_cand = min(n, 32);

    for (int iter = 0; iter < n + 2; ++iter) {
        if (n_cand == 0) break;
        // pivot = median of the offered candidates (absent lanes sort last)
        unsigned long long sk = cand_k;
        int si = cand_i;
        warp_sort_order(sk, si, lane);
        unsigned long long pv_k = __shfl_sync(0xffffffffu, sk, n_cand >> 1);
        int pv_i = __shfl_sync(0xffffffffu, si, n_cand >> 1);

        double mass_before = 0.0;
        unsigned long long ca_k = 0ull, cb_k = 0ull;
        int ca_i = 0x7fffffff, cb_i = 0x7fffffff;   // first element of each side seen by this lane
        for (int j = lane; j < n; j += 32) {
            unsigned long long kj = ek[j];
            if (!precedes(lo_k, lo_i, kj, j) || !precedes(kj, j, hi_k, hi_i)) continue;
            if (precedes(kj, j, pv_k, pv_i)) {
                mass_before += __longlong_as_double((long long)kj);
                if (ca_i == 0x7fffffff) { ca_k = kj; ca_i = j; }
            } else if (precedes(pv_k, pv_i, kj, j)) {
                if (cb_i == 0x7fffffff) { cb_k = kj; cb_i = j; }
            }
        }
        mass_before = warp_sum(mass_before);
        double pv_e = __longlong_as_double((long long)pv_k);
        if (base + mass_before >= target) {          // crossing strictly before the pivot
            hi_k = pv_k; hi_i = pv_i;
            cand_k = ca_k; cand_i = ca_i;
        } else if (base + mass_before + pv_e >= target) {
            return OrderKey{pv_k, pv_i};              // the pivot is the crossing element
        } else {
            base += mass_before + pv_e;
            lo_k = pv_k; lo_i = pv_i;
            cand_k = cb_k; cand_i = cb_i;
        }
        n_cand = __popc(__ballot_sync(0xffffffffu, cand_i != 0x7fffffff));
    }
    // Interval exhausted without reaching the target (rounding of partial sums): keep all up to hi.
    if (hi_i == 0x7fffffff) return OrderKey{0ull, 0x7fffffff};
    return OrderKey{lo_k, lo_i};
}

// One warp per query row of the chunk.  Writes the per-tile mask matrix (always) and the
// optional raster-ordered bitmap / count outputs.  dynamic smem: warps_per_cta * N_ld doubles.
__global__ void __launch_bounds__(128) select_kernel(Geom g, int gt0, int n_gt,
                                                     const double* __restrict__ logits,
                                                     uint32_t* __restrict__ tile_mask,
                                                     uint32_t* __restrict__ sel_bitmap,
                                                     int32_t* __restrict__ sel_count) {
    extern __shared__ double sel_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row_id = blockIdx.x * 4 + warp;        // row within the chunk
    if (row_id >= n_gt * kTileRows) return;
    const int gt = gt0 + row_id / kTileRows, r = row_id % kTileRows;
    const int tile = gt % g.n_tiles, bh = gt / g.n_tiles;
    const int h = bh % g.Hq, b = bh / g.Hq;
    const int pos = tile * kTileRows + r;
    double* e = sel_smem + (size_t)warp * g.N_ld;
    const double* s = logits + (size_t)row_id * g.N_ld;

    const int n = pos < g.S ? n_candidates(g, pos) : 0;
    OrderKey bd{0ull, 0x7fffffff};                  // default: everything precedes the boundary
    if (n > 0 && g.top_p < 1.0) {
        double mx = -INFINITY;
        for (int j = lane; j < n; j += 32) mx = fmax(mx, s[j]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        double z = 0.0;
        for (int j = lane; j < n; j += 32) {
            double ej = exp(s[j] - mx);
            e[j] = ej;
            z += ej;
        }
        z = warp_sum(z);
        __syncwarp();
        bd = nucleus_boundary(e, n, g.top_p * z, lane);
    } else {
        for (int j = lane; j < n; j += 32) e[j] = 1.0;
        __syncwarp();
    }

    const unsigned long long* ek = reinterpret_cast<const unsigned long long*>(e);
    const int raster = pos < g.S ? pos_to_raster(g, pos) : 0;
    int count = 0;
    for (int w = 0; w < g.n_words; ++w) {
        int j = w * 32 + lane;
        bool on = false;
        if (j < n) {
            unsigned long long kj = ek[j];
            on = !precedes(bd.key, bd.idx, kj, j);   // j precedes or equals the boundary
        }
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
