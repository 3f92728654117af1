// K4 (legacy tensor path): gathered flash-style attention with mma.sync.m16n8k16 (Eq. 3).
//
// Kept as the simple, independently written cross-check of the tcgen05 kernel and as the path
// for shapes the tcgen05 kernel does not take.  One CTA = one tile of 128 query rows (cube-major
// positions) of one query head; 8 warps x 16 rows.  Key/value blocks of 64 cube-major positions
// are visited if (a) any row of the tile selected a cube inside the block, or (b) the block
// overlaps the tile's local range (own cubes of video rows / text prefix of text rows).  Inside
// a visited block every (row, key) pair is masked by key_allowed(), so each row attends exactly
// its own key set although the tile iterates over the union.
#pragma once
#include "common.cuh"

namespace adaspark {

template <int D>
struct MmaAttnSmem {
    __nv_bfloat16 q[kTileRows][D];          // swizzled 16-byte chunks
    __nv_bfloat16 k[2][kBlockTok][D];       // [stage][token][d], swizzled
    __nv_bfloat16 vt[2][D][kBlockTok];      // [stage][d][token], swizzled
    uint32_t union_words[128];              // OR over the tile's rows of each selection word
};

// 16-byte chunk swizzle: rows of (8 * n_chunk_groups) chunks; chunk' = chunk ^ (row & 7).
__device__ __forceinline__ int swz(int row, int chunk) { return chunk ^ (row & 7); }

template <int D>
__global__ void __launch_bounds__(256) attn_prefill_mma_kernel(Geom g, const __nv_bfloat16* __restrict__ q,
                                                               const __nv_bfloat16* __restrict__ k_cube,
                                                               const __nv_bfloat16* __restrict__ v_cube,
                                                               const uint32_t* __restrict__ tile_mask,
                                                               __nv_bfloat16* __restrict__ out,
                                                               unsigned long long* __restrict__ executed_blocks) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    MmaAttnSmem<D>& sm = *reinterpret_cast<MmaAttnSmem<D>*>(smem_raw);
    constexpr int kQChunks = D / 8;   // 16-byte chunks per K/Q row
    constexpr int kKSteps = D / 16;   // k-steps of QK^T
    constexpr int kDTiles = D / 8;    // n-tiles of the output

    const int tile = g.n_tiles - 1 - blockIdx.x;  // long (late) tiles first
    const int h = blockIdx.y, b = blockIdx.z, gk = h / g.G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tile_pos0 = tile * kTileRows;
    const int tile_end = min(tile_pos0 + kTileRows, g.S);   // exclusive

    // ---- Q tile -> smem (gather rows from raster order)
    for (int idx = tid; idx < kTileRows * kQChunks; idx += 256) {
        int row = idx / kQChunks, c = idx - row * kQChunks;
        int pos = tile_pos0 + row;
        uint4 val = make_uint4(0, 0, 0, 0);
        if (slot_live(g, pos))
            val = *reinterpret_cast<const uint4*>(q + (io_row(g, b, pos) * g.Hq + h) * D + c * 8);
        *reinterpret_cast<uint4*>(&sm.q[row][swz(row, c) * 8]) = val;
    }
    // ---- union of the rows' selection words
    for (int w = warp; w < g.n_words; w += 8) {
        uint32_t u = 0;
        for (int r = lane; r < kTileRows; r += 32) u |= tile_mask[mask_index(g, b, h, tile, w, r)];
        u = __reduce_or_sync(0xffffffffu, u);
        if (lane == 0) sm.union_words[w] = u;
    }
    __syncthreads();

    // local range of the tile: from the first row's own cube (video) or the text start
    const int local_start = tile_pos0 < g.S_v ? (tile_pos0 / g.C) * g.C : g.S_v;
    const int first_local_blk = local_start / kBlockTok;
    // blocks up to the tile's own end, and for a tile with video rows also those of the text prefix
    const int n_blk_own = (tile_end + kBlockTok - 1) / kBlockTok;
    const bool sees_prefix = g.n_prefix > 0 && tile_pos0 < g.S_v;
    const int prefix_blk0 = g.S_v / kBlockTok;
    const int n_blk = sees_prefix ? max(n_blk_own, (g.S_v + g.n_prefix + kBlockTok - 1) / kBlockTok) : n_blk_own;

    auto block_needed = [&](int kb) -> bool {
        if (kb >= n_blk_own) return kb >= prefix_blk0;
        if (kb >= first_local_blk) return true;
        // cubes overlapping block kb: [kb*64 / C, (kb*64 + 63) / C]
        int c_lo = (kb * kBlockTok) / g.C, c_hi = (kb * kBlockTok + kBlockTok - 1) / g.C;
        uint32_t word = sm.union_words[c_lo >> 5];
        uint32_t span = c_hi - c_lo + 1;   // <= 4 cubes, never crosses a word (aligned)
        uint32_t bits = (span >= 32 ? 0xffffffffu : ((1u << span) - 1u)) << (c_lo & 31);
        return (word & bits) != 0;
    };
    auto next_block = [&](int kb) -> int {
        while (kb < n_blk && !block_needed(kb)) ++kb;
        return kb;
    };

    const __nv_bfloat16* kbase = k_cube + (size_t)(b * g.Hkv + gk) * g.S_cap * D;
    const __nv_bfloat16* vbase = v_cube + (size_t)(b * g.Hkv + gk) * g.n_kv_blocks_cap * D * kBlockTok;
    auto load_block = [&](int kb, int stage) {
        const __nv_bfloat16* ksrc = kbase + (size_t)kb * kBlockTok * D;
        for (int idx = tid; idx < kBlockTok * kQChunks; idx += 256) {
            int row = idx / kQChunks, c = idx - row * kQChunks;
            cp_async_16(&sm.k[stage][row][swz(row, c) * 8], ksrc + (size_t)row * D + c * 8);
        }
        const __nv_bfloat16* vsrc = vbase + (size_t)kb * D * kBlockTok;
        for (int idx = tid; idx < D * 8; idx += 256) {
            int row = idx >> 3, c = idx & 7;
            cp_async_16(&sm.vt[stage][row][swz(row, c) * 8], vsrc + (size_t)row * kBlockTok + c * 8);
        }
    };

    // ---- Q fragments (A operand, 16 rows x D per warp) stay in registers
    uint32_t qf[kKSteps][4];
    {
        int row = warp * 16 + (lane & 15);
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
            int chunk = ks * 2 + (lane >> 4);
            ldmatrix_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], &sm.q[row][swz(row, chunk) * 8]);
        }
    }

    const int rA = warp * 16 + (lane >> 2), rB = rA + 8;
    const int posA = tile_pos0 + rA, posB = tile_pos0 + rB;
    float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
    float o[kDTiles][4];
#pragma unroll
    for (int i = 0; i < kDTiles; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

    int kb = next_block(0);
    if (kb < n_blk) load_block(kb, 0);
    cp_async_commit();
    int stage = 0, visited = 0;
    while (kb < n_blk) {
        ++visited;
        int kb_next = next_block(kb + 1);
        if (kb_next < n_blk) load_block(kb_next, stage ^ 1);
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();

        // ---- S = Q K^T  (16 x 64 per warp)
        float s[8][4];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {   // pairs of 8-token n-tiles
                // matrices: (tokens np*16 + 0..7, d lo), (same tokens, d hi), (tokens +8, d lo), (+8, d hi)
                int row = np * 16 + (lane & 7) + ((lane >> 4) << 3);
                int chunk = ks * 2 + ((lane >> 3) & 1);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3, &sm.k[stage][row][swz(row, chunk) * 8]);
                mma_bf16_16816(s[np * 2], qf[ks], b0, b1);
                mma_bf16_16816(s[np * 2 + 1], qf[ks], b2, b3);
            }
        }

        // ---- mask + online softmax (base-2 domain)
        const int pk0 = kb * kBlockTok;
        uint32_t wordA = 0, wordB = 0;
        if (pk0 < g.S_v) {
            int w = (pk0 / g.C) >> 5;
            wordA = tile_mask[mask_index(g, b, h, tile, w, rA)];
            wordB = tile_mask[mask_index(g, b, h, tile, w, rB)];
        }
        float mxA = -INFINITY, mxB = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                int pk = pk0 + nt * 8 + 2 * (lane & 3) + e;
                float va = key_allowed(g, posA, pk, wordA) ? s[nt][e] * g.scale_log2 : -INFINITY;
                float vb = key_allowed(g, posB, pk, wordB) ? s[nt][2 + e] * g.scale_log2 : -INFINITY;
                s[nt][e] = va;
                s[nt][2 + e] = vb;
                mxA = fmaxf(mxA, va);
                mxB = fmaxf(mxB, vb);
            }
        }
        mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 1));
        mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 2));
        mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 1));
        mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 2));
        float mA_new = fmaxf(mA, mxA), mB_new = fmaxf(mB, mxB);
        float refA = (mA_new == -INFINITY) ? 0.f : mA_new;   // rows with nothing visible yet
        float refB = (mB_new == -INFINITY) ? 0.f : mB_new;
        float corrA = fast_exp2(mA - refA), corrB = fast_exp2(mB - refB);
        mA = mA_new;
        mB = mB_new;
        float sumA = 0.f, sumB = 0.f;
        uint32_t pf[4][4];   // P as A fragments: 4 k-steps of 16 tokens
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            float p0 = fast_exp2(s[nt][0] - refA), p1 = fast_exp2(s[nt][1] - refA);
            float p2 = fast_exp2(s[nt][2] - refB), p3 = fast_exp2(s[nt][3] - refB);
            sumA += p0 + p1;
            sumB += p2 + p3;
            // A fragment of k-step kt = nt/2: regs {rowA k-lo, rowB k-lo, rowA k-hi, rowB k-hi}
            pf[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16x2(p0, p1);
            pf[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16x2(p2, p3);
        }
        lA = lA * corrA + sumA;
        lB = lB * corrB + sumB;
#pragma unroll
        for (int dt = 0; dt < kDTiles; ++dt) {
            o[dt][0] *= corrA; o[dt][1] *= corrA;
            o[dt][2] *= corrB; o[dt][3] *= corrB;
        }

        // ---- O += P V   (B operand from V^T: rows = d, 16-byte chunks of 8 tokens)
#pragma unroll
        for (int kt = 0; kt < 4; ++kt) {
#pragma unroll
            for (int dp = 0; dp < kDTiles / 2; ++dp) {   // pairs of 8-wide d tiles
                int row = dp * 16 + (lane & 7) + ((lane >> 4) << 3);
                int chunk = kt * 2 + ((lane >> 3) & 1);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3, &sm.vt[stage][row][swz(row, chunk) * 8]);
                mma_bf16_16816(o[dp * 2], pf[kt], b0, b1);
                mma_bf16_16816(o[dp * 2 + 1], pf[kt], b2, b3);
            }
        }
        __syncthreads();   // all warps done with this stage before it is refilled
        stage ^= 1;
        kb = kb_next;
    }
    cp_async_wait<0>();
    if (tid == 0) atomicAdd(executed_blocks, (unsigned long long)visited);

    // ---- normalise and store at the raster position
    lA += __shfl_xor_sync(0xffffffffu, lA, 1);
    lA += __shfl_xor_sync(0xffffffffu, lA, 2);
    lB += __shfl_xor_sync(0xffffffffu, lB, 1);
    lB += __shfl_xor_sync(0xffffffffu, lB, 2);
    float invA = lA > 0.f ? 1.f / lA : 0.f, invB = lB > 0.f ? 1.f / lB : 0.f;
    if (slot_live(g, posA)) {
        __nv_bfloat16* dst = out + (io_row(g, b, posA) * g.Hq + h) * D + 2 * (lane & 3);
#pragma unroll
        for (int dt = 0; dt < kDTiles; ++dt)
            *reinterpret_cast<uint32_t*>(dst + dt * 8) = pack_bf16x2(o[dt][0] * invA, o[dt][1] * invA);
    }
    if (slot_live(g, posB)) {
        __nv_bfloat16* dst = out + (io_row(g, b, posB) * g.Hq + h) * D + 2 * (lane & 3);
#pragma unroll
        for (int dt = 0; dt < kDTiles; ++dt)
            *reinterpret_cast<uint32_t*>(dst + dt * 8) = pack_bf16x2(o[dt][2] * invB, o[dt][3] * invB);
    }
}

}  // namespace adaspark
