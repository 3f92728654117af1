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
//   select_kernel  G lanes per query row (8, 16 or 32 by the number of cubes): exact fixed-point
//                  softmax masses, radix selection of the nucleus boundary (select_radix.cuh, no
//                  sort), then ballots emit the row's bitmap words.
#pragma once
#include "common.cuh"
#include "select_radix.cuh"

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

// G lanes per query row of the chunk, 32/G rows per warp.  Writes the per-tile mask matrix (always)
// and the optional raster-ordered bitmap / count outputs.  Short rows (G < 32) keep their order keys
// in shared memory; long rows (G = 32) overwrite their scores in the L2-resident score buffer with
// the keys, so that shared memory per warp stays small and many warps hide the latency of the passes.
// dynamic smem per warp: kSelHistWords + (32/G) * (keys in smem ? N_ld : 0 + cand_cap) words of 8 bytes.
constexpr int kSelectWarps = 1;     // one-warp CTAs pack shared memory best (measured)
__host__ __device__ inline int select_lanes_per_row(int N_ld) { return N_ld <= 256 ? 8 : (N_ld <= 512 ? 16 : 32); }
__host__ __device__ inline int select_cand_cap(int N_ld) { return N_ld <= 256 ? 64 : (N_ld <= 512 ? 128 : (N_ld <= 1024 ? 256 : 512)); }
__host__ __device__ inline size_t select_smem_bytes(int N_ld) {
    const int rows = 32 / select_lanes_per_row(N_ld);
    const int lanes = select_lanes_per_row(N_ld);
    return (size_t)kSelectWarps * ((size_t)kSelHistWords + (size_t)rows * ((lanes < 32 ? N_ld : 0) + select_cand_cap(N_ld))) * 8;
}

template <int G>
__global__ void __launch_bounds__(kSelectWarps * 32) select_kernel(Geom g, int gt0, int n_gt,
                                                                   double* logits,
                                                                   uint32_t* __restrict__ tile_mask,
                                                                   uint32_t* __restrict__ sel_bitmap,
                                                                   int32_t* __restrict__ sel_count) {
    extern __shared__ __align__(16) unsigned long long sel_smem[];
    constexpr int kRows = SelGeom<G>::kRows;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int gi = lane / G, gl = lane & (G - 1), gbase = lane & ~(G - 1);
    const int row0 = (blockIdx.x * kSelectWarps + warp) * kRows;      // first row of the warp within the chunk
    if (row0 >= n_gt * kTileRows) return;
    const int cand_cap = select_cand_cap(g.N_ld);
    constexpr bool kInPlace = (G == 32);
    const int key_words = kInPlace ? 0 : g.N_ld;
    const size_t per_warp = (size_t)kSelHistWords + (size_t)kRows * (key_words + cand_cap);
    unsigned long long* hist = sel_smem + (size_t)warp * per_warp;
    unsigned long long* cand = hist + kSelHistWords + (size_t)kRows * key_words + (size_t)gi * cand_cap;

    // the rows of a warp lie in one query tile (kRows divides 128)
    const int gt = gt0 + row0 / kTileRows, r = row0 % kTileRows + gi;
    int tile, bh, h, b;
    g.div_n_tiles.divmod(gt, bh, tile);
    g.div_Hq.divmod(bh, b, h);
    const int pos = tile * kTileRows + r;
    double* s = logits + (size_t)(row0 + gi) * g.N_ld;
    unsigned long long* keys = kInPlace ? reinterpret_cast<unsigned long long*>(s) : hist + kSelHistWords + (size_t)gi * g.N_ld;

    const int n = pos < g.S ? n_candidates(g, pos) : 0;
    const bool all = g.top_k <= 0 && !(g.top_p < 1.0);
    unsigned long long bd = 0ull;                    // 0: every candidate is selected
    if (!all) bd = nucleus_boundary_radix<G, kInPlace>(s, n, g.top_p, g.top_k, keys, hist, cand, cand_cap, lane);

    const bool extra = (sel_bitmap != nullptr || sel_count != nullptr) && pos < g.S;
    const int raster = extra ? pos_to_raster(g, pos) : 0;
    int count = 0;
    for (int w = 0; w < g.n_words; ++w) {
        uint32_t word = 0;
#pragma unroll
        for (int k = 0; k < 32 / G; ++k) {           // bit k*G + gl of the word
            const int j = w * 32 + k * G + gl;
            const bool on = j < n && (all || keys[j] >= bd);
            const uint32_t ball = __ballot_sync(0xffffffffu, on);
            word |= (G == 32 ? ball : ((ball >> gbase) & ((1u << G) - 1u))) << (k * G);
        }
        count += __popc(word);
        if (gl == 0) {
            tile_mask[mask_index(g, b, h, tile, w, r)] = word;
            if (sel_bitmap && extra)
                sel_bitmap[((size_t)(b * g.Hq + h) * g.S + raster) * g.n_words + w] = word;
        }
    }
    if (sel_count && gl == 0 && extra) sel_count[(size_t)(b * g.Hq + h) * g.S + raster] = count;
}

}  // namespace adaspark
