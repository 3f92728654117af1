// K3, fp64 path: cube scoring (Eq. 1) and nucleus selection (Eq. 2) of single query rows on the
// CUDA cores, one warp per row.  Every product bf16 x fp32 is exact in fp64 and the sums are fp64, so
// this path has no input-range assumption.  It serves
//   - the rows the tensor-core kernel (score_select_fused.cuh) hands over: rows whose exponents
//     are outside its validated range, rows with more exactly tied cubes at the nucleus boundary than
//     it can hold, rows it gave up on (list mode: row ids from the workspace, count read on the device);
//   - every row, as the independent cross-check path of the library (all mode).
// Per row: the lanes compute the scores of cubes lane, lane + 32, ... into a scratch row in global
// memory (L2-resident), the radix routine of select_radix.cuh finds the boundary key in place, ballots
// emit the row's words, and the words are OR-ed into the tile's union.
#pragma once
#include "common.cuh"
#include "select_radix.cuh"

namespace adaspark {

constexpr int kExactWarps = 4;          // warps (rows in flight) per CTA
constexpr int kExactCandCap = 256;

// rows: nullptr = all mode (row id runs over [0, n_ids)); else list mode, n_ids is ignored and
// *n_list rows are taken from rows[].  Row id = ((b*Hq + h)*n_tiles_cap + tile)*128 + r.
// scratch: gridDim.x * kExactWarps rows of N_ld doubles.
template <int D>
__global__ void __launch_bounds__(kExactWarps * 32) select_exact_kernel(
    Geom g, const __nv_bfloat16* __restrict__ q, const float* __restrict__ cube_keys, const int32_t* __restrict__ rows,
    const uint32_t* __restrict__ n_list, long long n_ids, double* __restrict__ scratch, uint32_t* __restrict__ tile_mask,
    uint32_t* __restrict__ tile_union, uint32_t* __restrict__ sel_bitmap, int32_t* __restrict__ sel_count) {
    __shared__ __align__(16) unsigned long long hist_s[kExactWarps][kSelHistWords + kExactCandCap];
    __shared__ double q_s[kExactWarps][D];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long total = rows ? (long long)*n_list : n_ids;
    const long long stride = (long long)gridDim.x * kExactWarps;
    double* s = scratch + ((size_t)blockIdx.x * kExactWarps + warp) * g.N_ld;
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(s);
    unsigned long long* hist = hist_s[warp];
    double* qd = q_s[warp];
    const bool all = g.top_k <= 0 && !(g.top_p < 1.0);

    for (long long idx = (long long)blockIdx.x * kExactWarps + warp; idx < total; idx += stride) {
        const long long id = rows ? (long long)rows[idx] : idx;
        const int r = (int)(id & (kTileRows - 1));
        const int gt_cap = (int)(id >> 7);
        const int bh = gt_cap / g.n_tiles_cap, tile = gt_cap - bh * g.n_tiles_cap;
        if (tile >= g.n_tiles || tile < g.tile_begin) continue;
        int b, h;
        g.div_Hq.divmod(bh, b, h);
        const int gk = h / g.G;
        const int pos = tile * kTileRows + r;
        const bool live = slot_live(g, pos);
        const int n = live ? n_candidates(g, pos) : 0;
        const int raster = live ? pos_to_io(g, pos) - g.pos_begin : 0;   // row of the call's tensors
        unsigned long long bd = 0ull;                    // 0: every candidate is selected
        if (!all && n > 0) {
            // ---- scores: s[j] = scale * <q, kbar_j> in fp64
            const __nv_bfloat16* qsrc = q + (((size_t)b * g.S_io + raster) * g.Hq + h) * D;
            for (int d = lane; d < D; d += 32) qd[d] = (double)__bfloat162float(qsrc[d]);
            __syncwarp();
            const float* kbase = cube_keys + (size_t)(b * g.Hkv + gk) * g.N * D;
            for (int j = lane; j < n; j += 32) {
                const float4* kr = reinterpret_cast<const float4*>(kbase + (size_t)j * D);
                double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
#pragma unroll 8
                for (int d4 = 0; d4 < D / 4; ++d4) {
                    const float4 kv = __ldg(kr + d4);
                    a0 = fma(qd[4 * d4 + 0], (double)kv.x, a0);
                    a1 = fma(qd[4 * d4 + 1], (double)kv.y, a1);
                    a2 = fma(qd[4 * d4 + 2], (double)kv.z, a2);
                    a3 = fma(qd[4 * d4 + 3], (double)kv.w, a3);
                }
                s[j] = ((a0 + a1) + (a2 + a3)) * g.scale_d;
            }
            __syncwarp();
            bd = nucleus_boundary_radix<32, true>(s, n, g.top_p, g.top_k, keys, hist, hist + kSelHistWords, kExactCandCap, lane);
        }
        // ---- the row's words
        const bool extra = live && (sel_bitmap != nullptr || sel_count != nullptr);
        int count = 0;
        for (int w = 0; w < g.n_words; ++w) {
            const int j = w * 32 + lane;
            const bool on = j < n && (all || keys[j] >= bd);
            const uint32_t word = __ballot_sync(0xffffffffu, on);
            count += __popc(word);
            if (lane == 0) {
                tile_mask[mask_index(g, b, h, tile, w, r)] = word;
                if (word) atomicOr(tile_union + (size_t)gt_cap * g.n_words + w, word);
                if (sel_bitmap && extra) sel_bitmap[((size_t)(b * g.Hq + h) * g.S_io + raster) * g.n_words + w] = word;
            }
        }
        if (sel_count && lane == 0 && extra) sel_count[(size_t)(b * g.Hq + h) * g.S_io + raster] = count;
        __syncwarp();
    }
}

}  // namespace adaspark
