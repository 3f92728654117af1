// K3 on the bf16 tensor cores: cube scores of Eq. 1 from error-free digit slices.
//
// The selection must follow an fp64 evaluation of Eqs. 1-2 (rows may differ only inside a 1e-6
// probability margin), so plain bf16/fp32 tensor-core arithmetic is not accurate enough.  Instead
// every query row q and every mean key k are written in fixed point relative to the largest
// exponent of their row,
//     x = 2^(e - 30) * (d0*2^24 + d1*2^16 + d2*2^8 + d3),   digits d_i integers in [-128, 128],
// (exact for elements within 2^-23 (q, 8 significant bits) / 2^-7 (k, 24 bits) of the row maximum,
// rounded at 2^-30 of it below that).  Digits are exact bf16 values, a product of two digits has 15
// bits and a sum of 4 * 128 such products stays below 2^24, so a tcgen05.mma with fp32 accumulation
// computes  S_L = sum_{a+b=L} Q_a . K_b  EXACTLY for each level L.  Then
//     q . k = 2^(e_q + e_k - 12) * (S_0 + S_1*2^-8 + S_2*2^-16 + S_3*2^-24 + levels >= 4),
// and the levels 0..3 (10 digit pairs, four TMEM accumulators) are combined exactly in fp64.  The
// dropped levels are bounded by 1.5e-3 * 2^-12 * 2^(e_q+e_k) in the worst case (all digit products
// aligned), about 5e-7 in the scaled logit for |q| <= 3, |k| <= 5 and typically 10x less: inside
// the margin above.
//
//   slice_keys_kernel   digit planes + row exponents of the mean keys (once per forward, tiny)
//   score_tc_kernel     persistent CTAs, one per SM; work item = one 128-row query tile x a group of
//                       64-cube column tiles.  Roles (448 threads), pipelined across items:
//     warps 0-3   epilogue (thread = row = TMEM lane): TMEM -> fp64 scores -> coalesced rows of the
//                 score buffer.  The four level accumulators are double-buffered in TMEM (2 x 4 x 64
//                 columns), so the epilogue of one column tile overlaps the MMAs of the next
//     warps 4-11  slicers (two threads per row): read the bf16 query row, compute its digits in
//                 registers while the previous item's MMAs still read the planes, then store the
//                 four swizzled digit planes of the tile into shared memory
//     warp 12     TMA producer: key digit blocks (plane, 64-d panel, 64 cubes) in a ring
//     warp 13     issues the tcgen05.mma stream (80 of 128x64x16 per column tile at D = 128)
#pragma once
#include "tc_common.cuh"

namespace adaspark {

constexpr int kScoreTcThreads = 448;
constexpr int kScoreTcRing = 8;          // key digit blocks (64 cubes x 64 d, 8 KB) in flight
constexpr int kScoreTcCols = 64;         // cubes per column tile

// Fixed-point value of x relative to the row exponent e (unbiased exponent of the row maximum):
// round(x * 2^(30 - e)), |result| < 2^31.
__device__ __forceinline__ int fixed30(float x, int e) {
    return __float2int_rn(x * __int_as_float((157 - e) << 23));   // 2^(30 - e), exact for e >= -96
}
// Signed base-256 digits, most significant first: v = d[0]*2^24 + d[1]*2^16 + d[2]*2^8 + d[3].
__device__ __forceinline__ void digits256(int v, int (&d)[4]) {
    // v = 256 * (floor(v / 256) + carry) + digit with digit = low byte read as signed (no overflow)
    d[3] = (int)(signed char)(v & 0xff);
    v = (v >> 8) + (d[3] < 0 ? 1 : 0);
    d[2] = (int)(signed char)(v & 0xff);
    v = (v >> 8) + (d[2] < 0 ? 1 : 0);
    d[1] = (int)(signed char)(v & 0xff);
    d[0] = (v >> 8) + (d[1] < 0 ? 1 : 0);
}
// The same digits for a float that holds an integer-valued (or nearly: |fraction| only in the last
// digit) fixed-point number v, |v| < 2^31, computed with exact float operations.
__device__ __forceinline__ float round_small(float t) {          // nearest integer, |t| <= 2^22
    return (t + 12582912.f) - 12582912.f;
}
__device__ __forceinline__ void float_digits256(float v, float (&d)[4]) {
    d[0] = round_small(v * (1.f / 16777216.f));
    float r = fmaf(-d[0], 16777216.f, v);
    d[1] = round_small(r * (1.f / 65536.f));
    r = fmaf(-d[1], 65536.f, r);
    d[2] = round_small(r * (1.f / 256.f));
    r = fmaf(-d[2], 256.f, r);
    d[3] = round_small(r);
}
// bf16 bit pattern of a small integer (|i| <= 256: exact).
__device__ __forceinline__ uint32_t bf16_bits_of_int(int i) {
    return __float_as_uint((float)i) >> 16;
}
__device__ __forceinline__ int exponent_of(float x) {   // unbiased exponent field (0 for zero/denormal rows)
    const int e = (int)((__float_as_uint(x) >> 23) & 0xffu);
    return e == 0 ? 0 : max(e - 127, -90);     // rows smaller than 2^-90 keep fewer digits
}

// Digit planes of the mean keys: planes[p][(b*Hkv+gk)*N_ld + cube][D] (bf16), key_exp[(b*Hkv+gk)*N_ld + cube].
// One warp per cube row; rows >= N inside the padded leading dimension are zero-filled.
__global__ void __launch_bounds__(128) slice_keys_kernel(Geom g, const float* __restrict__ cube_keys,
                                                         __nv_bfloat16* __restrict__ planes, int32_t* __restrict__ key_exp) {
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5);              // (b*Hkv+gk)*N_ld + cube
    const int n_rows = g.B * g.Hkv * g.N_ld;
    if (row >= n_rows) return;
    const int bh = row / g.N_ld, cube = row - bh * g.N_ld;
    const size_t plane_stride = (size_t)n_rows * g.D;
    const bool live = cube < g.N;
    const float* src = cube_keys + ((size_t)bh * g.N + (live ? cube : 0)) * g.D;
    float mx = 0.f;
    for (int d = lane; d < g.D; d += 32) mx = fmaxf(mx, live ? fabsf(src[d]) : 0.f);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const int e = exponent_of(mx);
    for (int d = lane; d < g.D; d += 32) {
        int dg[4];
        digits256(live ? fixed30(src[d], e) : 0, dg);
#pragma unroll
        for (int p = 0; p < 4; ++p)
            planes[p * plane_stride + (size_t)row * g.D + d] = __ushort_as_bfloat16((unsigned short)bf16_bits_of_int(dg[p]));
    }
    if (lane == 0) key_exp[row] = e;
}

template <int D>
struct ScoreTcSmem {
    __nv_bfloat16 qd[4][D / 64][128][64];               // digit planes of the Q tile, UMMA layout (128-B swizzle)
    __nv_bfloat16 kring[kScoreTcRing][kScoreTcCols][64];   // key digit blocks: [cube][64 d of one panel of one plane]
    double stage[128][32];                              // epilogue: scores of 32 columns, column index ^ (row & 31)
    uint64_t q_sliced, qd_free, k_full[kScoreTcRing], k_group_empty[kScoreTcRing / 4], acc_full[2], acc_free[2];
    uint32_t tmem_base;
    int abort_flag;
};

// Work item `it` of the launch: query tile gt0 + it / groups, column tiles [ct0, ct1).
struct ScoreItem {
    int b, h, gk, tile, ct0, ct1, tile_in_chunk;
};
__device__ __forceinline__ ScoreItem score_item(const Geom& g, int gt0, int groups, int cols_per_cta, int it) {
    ScoreItem w;
    w.tile_in_chunk = it / groups;
    const int grp = it - w.tile_in_chunk * groups;
    int bh;
    g.div_n_tiles.divmod(gt0 + w.tile_in_chunk, bh, w.tile);
    g.div_Hq.divmod(bh, w.b, w.h);
    w.gk = w.h / g.G;
    const int last_pos = min(w.tile * kTileRows + kTileRows, g.S) - 1;
    const int n_ct = (n_candidates(g, last_pos) + kScoreTcCols - 1) / kScoreTcCols;
    w.ct0 = grp * cols_per_cta;
    w.ct1 = min(w.ct0 + cols_per_cta, n_ct);          // ct0 >= ct1: nothing to do for this item
    return w;
}

// grid = min(items, SMs) persistent CTAs.  logits: the chunk's score buffer,
// logits[(tile_in_chunk*128 + r) * N_ld + j] = scale * <q_row, kbar_j>.  q_cube: cube-major bf16 queries
// [B*Hq, S_cap, D].
template <int D>
__global__ void __launch_bounds__(kScoreTcThreads, 1) score_tc_kernel(
    Geom g, int gt0, int n_items, int groups, int cols_per_cta, const __nv_bfloat16* __restrict__ q_cube,
    const __grid_constant__ CUtensorMap tmK, const int32_t* __restrict__ key_exp, double* __restrict__ logits,
    int32_t* __restrict__ status) {
    extern __shared__ unsigned char score_tc_raw[];
    ScoreTcSmem<D>& sm = *reinterpret_cast<ScoreTcSmem<D>*>((reinterpret_cast<uintptr_t>(score_tc_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kPanels = D / 64;
    constexpr int kBlocks = 4 * kPanels;                          // key digit blocks per column tile
    constexpr uint32_t kIdesc = tc::make_idesc_bf16(128, kScoreTcCols);
    constexpr uint32_t kBlockBytes = kScoreTcCols * 64 * 2;
    constexpr int kProducerWarp = 12, kMmaWarp = 13;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        tc::mbar_init(&sm.q_sliced, 256);
        tc::mbar_init(&sm.qd_free, 1);
        for (int i = 0; i < kScoreTcRing; ++i) {
            tc::mbar_init(&sm.k_full[i], 1);
        }
        // a tcgen05.commit costs about two MMA slots: the ring is released four blocks (one panel's
        // digit planes) at a time
        for (int i = 0; i < kScoreTcRing / 4; ++i) tc::mbar_init(&sm.k_group_empty[i], 1);
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(&sm.acc_full[i], 1);
            tc::mbar_init(&sm.acc_free[i], 128);
        }
        sm.abort_flag = 0;
        tc::fence_barrier_init();
    }
    if (warp == kProducerWarp) {
        tc::tmem_alloc<512>(&sm.tmem_base);
        if (lane == 0) tc::prefetch_tensormap(&tmK);
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tbase = sm.tmem_base;
    volatile int* abort_flag = &sm.abort_flag;

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const int n_rows = g.B * g.Hkv * g.N_ld;
            int i = 0;                                            // running block counter of this CTA
            bool ok = true;
            for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x) {
                const ScoreItem w = score_item(g, gt0, groups, cols_per_cta, it);
                const int k_row0 = (w.b * g.Hkv + w.gk) * g.N_ld;
                for (int ct = w.ct0; ok && ct < w.ct1; ++ct) {
                    for (int blk = 0; blk < kBlocks; ++blk, ++i) {
                        const int p = blk >> 2, plane = blk & 3, s = i % kScoreTcRing, u = i / kScoreTcRing;
                        if ((blk & 3) == 0 && !(ok = tc::mbar_wait(&sm.k_group_empty[s >> 2], (u & 1) ^ 1, abort_flag))) break;
                        tc::mbar_arrive_expect_tx(&sm.k_full[s], kBlockBytes);
                        tc::tma_load_2d(&sm.kring[s][0][0], &tmK, p * 64, plane * n_rows + k_row0 + ct * kScoreTcCols, &sm.k_full[s]);
                    }
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t kPlaneStep = (uint32_t)sizeof(sm.qd[0]) >> 4, kPanelStep = (128 * 64 * 2) >> 4;
            constexpr uint32_t kRingStep = (uint32_t)sizeof(sm.kring[0]) >> 4, kKStep = 32 >> 4;
            const uint32_t q_lo0 = tc::smem_desc_lo_sw128(smem_u32(&sm.qd[0][0][0][0]));
            const uint32_t k_lo0 = tc::smem_desc_lo_sw128(smem_u32(&sm.kring[0][0][0]));
            bool ok = true;
            int i = 0, c = 0, n_done = 0;                         // running block / column-tile / item counters
            for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x) {
                const ScoreItem w = score_item(g, gt0, groups, cols_per_cta, it);
                if (w.ct0 >= w.ct1) continue;
                if (!(ok = tc::mbar_wait(&sm.q_sliced, n_done & 1, abort_flag))) break;
                for (int ct = w.ct0; ok && ct < w.ct1; ++ct, ++c) {
                    const int buf = c & 1, use = c >> 1;          // accumulator set and how often it was used before
                    if (use > 0 && !(ok = tc::mbar_wait(&sm.acc_free[buf], (use - 1) & 1, abort_flag))) break;
                    tc::tc_fence_after_sync();
                    for (int blk = 0; blk < kBlocks; ++blk, ++i) {
                        const int p = blk >> 2, plane = blk & 3, s = i % kScoreTcRing, u = i / kScoreTcRing;
                        if (!(ok = tc::mbar_wait(&sm.k_full[s], u & 1, abort_flag))) break;
                        tc::tc_fence_after_sync();
                        const uint32_t kb = k_lo0 + s * kRingStep;
                        for (int a = 0; a + plane <= 3; ++a) {    // level a + plane
                            const uint32_t qa = q_lo0 + a * kPlaneStep + p * kPanelStep;
                            const uint32_t dst = tbase + buf * 256 + (a + plane) * kScoreTcCols;
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)
                                tc::umma_ss(dst, tc::smem_desc_from_halves(qa + ks * kKStep, tc::kSmemDescHiSw128),
                                            tc::smem_desc_from_halves(kb + ks * kKStep, tc::kSmemDescHiSw128), kIdesc,
                                            !(blk == 0 && ks == 0));
                        }
                        if ((blk & 3) == 3) tc::umma_commit(&sm.k_group_empty[s >> 2]);
                    }
                    if (ok) tc::umma_commit(&sm.acc_full[buf]);
                }
                if (ok) tc::umma_commit(&sm.qd_free);             // the digit planes may be overwritten
                ++n_done;
            }
        }
    } else if (warp >= 4) {
        // ------------------------------------------------------------ slicers (two threads per row)
        constexpr int kChunks = D / 16;                           // 16-byte chunks (8 elements) per thread
        const int r = (tid - 128) >> 1, half = (tid - 128) & 1;
        bool ok = true;
        int n_done = 0;
        for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x) {
            const ScoreItem w = score_item(g, gt0, groups, cols_per_cta, it);
            if (w.ct0 >= w.ct1) continue;
            const int pos = w.tile * kTileRows + r;
            const uint4* src = reinterpret_cast<const uint4*>(q_cube + ((size_t)(w.b * g.Hq + w.h) * g.S_cap + pos) * D) + half * kChunks;
            uint4 v[kChunks];
#pragma unroll
            for (int c = 0; c < kChunks; ++c) v[c] = pos < g.S ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);
            uint32_t mxbits = 0;
#pragma unroll
            for (int c = 0; c < kChunks; ++c) {
                const uint32_t wd[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
#pragma unroll
                for (int i = 0; i < 4; ++i) mxbits = max(mxbits, max(wd[i] & 0x7fffu, (wd[i] >> 16) & 0x7fffu));
            }
            mxbits = max(mxbits, __shfl_xor_sync(0xffffffffu, mxbits, 1));   // the two halves of the row
            const int ef = (int)(mxbits >> 7);
            const int e_q = ef == 0 ? 0 : max(ef - 127, -90);
            // digits in the float domain (every intermediate is exact): x * 2^(30-e) = d0*2^24 + d1*2^16 + d2*2^8 + d3
            const float mult = __int_as_float((157 - e_q) << 23);
            uint4 out[4][kChunks];
#pragma unroll
            for (int c = 0; c < kChunks; ++c) {
                const uint32_t wd[4] = {v[c].x, v[c].y, v[c].z, v[c].w};
                uint32_t pk[4][4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float dl[4], dh[4];
                    float_digits256(__uint_as_float(wd[i] << 16) * mult, dl);
                    float_digits256(__uint_as_float(wd[i] & 0xffff0000u) * mult, dh);
#pragma unroll
                    for (int pl = 0; pl < 4; ++pl)    // bf16 of a small integer = upper half of its float
                        pk[pl][i] = __byte_perm(__float_as_uint(dl[pl]), __float_as_uint(dh[pl]), 0x7632);
                }
#pragma unroll
                for (int pl = 0; pl < 4; ++pl) out[pl][c] = make_uint4(pk[pl][0], pk[pl][1], pk[pl][2], pk[pl][3]);
            }
            // the previous item's MMAs must have finished reading the digit planes
            if (n_done > 0 && !(ok = tc::mbar_wait(&sm.qd_free, (n_done - 1) & 1, abort_flag))) break;
            unsigned char* dst = reinterpret_cast<unsigned char*>(&sm.qd[0][0][0][0]);
#pragma unroll
            for (int c = 0; c < kChunks; ++c) {
                const int cc = half * kChunks + c;                // chunk of the row: panel cc / 8, position cc % 8
                const int off = (cc >> 3) * (128 * 128) + sw128(r, cc & 7);
#pragma unroll
                for (int pl = 0; pl < 4; ++pl) *reinterpret_cast<uint4*>(dst + (size_t)pl * sizeof(sm.qd[0]) + off) = out[pl][c];
            }
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // digit planes visible to the tensor core
            tc::mbar_arrive(&sm.q_sliced);
            ++n_done;
        }
    } else {
        // ------------------------------------------------------------ epilogue (thread = row = TMEM lane)
        const int r = tid;
        const uint32_t lane_addr = tbase + ((uint32_t)(warp * 32) << 16);
        bool ok = true;
        int c_run = 0, n_done = 0;
        for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x) {
            const ScoreItem w = score_item(g, gt0, groups, cols_per_cta, it);
            if (w.ct0 >= w.ct1) continue;
            // row exponent, recomputed from the query row exactly as the slicers do (the epilogue may
            // lag the slicers by more than one item, so nothing is handed over through shared memory)
            int e_q = 0;
            {
                const int pos = w.tile * kTileRows + r;
                const uint4* src = reinterpret_cast<const uint4*>(q_cube + ((size_t)(w.b * g.Hq + w.h) * g.S_cap + pos) * D);
                uint32_t mxbits = 0;
                if (pos < g.S) {
#pragma unroll
                    for (int c = 0; c < D / 8; ++c) {
                        const uint4 v = __ldg(src + c);
                        const uint32_t wd[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                        for (int i = 0; i < 4; ++i) mxbits = max(mxbits, max(wd[i] & 0x7fffu, (wd[i] >> 16) & 0x7fffu));
                    }
                }
                const int ef = (int)(mxbits >> 7);
                e_q = ef == 0 ? 0 : max(ef - 127, -90);
            }
            const double rowf = __hiloint2double((1023 + e_q) << 20, 0);          // 2^e_q
            const int32_t* kexp = key_exp + (size_t)(w.b * g.Hkv + w.gk) * g.N_ld;
            double* out_rows = logits + (size_t)w.tile_in_chunk * kTileRows * g.N_ld;
            for (int ct = w.ct0; ok && ct < w.ct1; ++ct, ++c_run) {
                const int buf = c_run & 1;
                if (!(ok = tc::mbar_wait(&sm.acc_full[buf], (c_run >> 1) & 1, abort_flag))) break;
                tc::tc_fence_after_sync();
#pragma unroll 1
                for (int c = 0; c < kScoreTcCols / 32; ++c) {     // 32 columns at a time through the staging tile
                    const int col0 = ct * kScoreTcCols + c * 32;
                    // column factor 2^(e_k - 36) * scale, held by the lane that owns the column
                    const int jc = col0 + lane;
                    const int ek = jc < g.N_ld ? kexp[jc] : 0;
                    const double colf = __hiloint2double((1023 + ek - 36) << 20, 0) * g.scale_d;
#pragma unroll
                    for (int hc = 0; hc < 2; ++hc) {
                        uint32_t lv[4][16];
#pragma unroll
                        for (int L = 0; L < 4; ++L) tc::tmem_ld_32x16(lane_addr + buf * 256 + L * kScoreTcCols + c * 32 + hc * 16, lv[L]);
                        tc::tmem_wait_ld();
                        if (c == kScoreTcCols / 32 - 1 && hc == 1) {   // last read of this accumulator set: release it
                            tc::tc_fence_before_sync();
                            tc::mbar_arrive(&sm.acc_free[buf]);
                        }
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            // exact integer level sums: S0*2^24 + S1*2^16 + S2*2^8 + S3 = hi*2^16 + lo
                            const int hi = __float2int_rn(__uint_as_float(lv[0][i])) * 256 + __float2int_rn(__uint_as_float(lv[1][i]));
                            const int lo = __float2int_rn(__uint_as_float(lv[2][i])) * 256 + __float2int_rn(__uint_as_float(lv[3][i]));
                            const double hd = __hiloint2double(0x43300000, hi ^ 0x80000000) - 4503601774854144.0;   // (double)hi
                            const double ld = __hiloint2double(0x43300000, lo ^ 0x80000000) - 4503601774854144.0;   // 2^52 + 2^31
                            const double v = fma(hd, 65536.0, ld);
                            const int col = hc * 16 + i;
                            const double cf = __shfl_sync(0xffffffffu, colf, col);
                            sm.stage[r][col ^ (r & 31)] = (v * rowf) * cf;
                        }
                    }
                    __syncwarp();
                    if (col0 + lane < g.N_ld) {
                        for (int rr = 0; rr < 32; ++rr) {
                            const int row = warp * 32 + rr;
                            out_rows[(size_t)row * g.N_ld + col0 + lane] = sm.stage[row][lane ^ (row & 31)];
                        }
                    }
                    __syncwarp();
                }
            }
            ++n_done;
        }
    }
    // ---------------------------------------------------------------- teardown
    tc::tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && sm.abort_flag) atomicExch(status, 6);
    if (warp == kProducerWarp) tc::tmem_dealloc<512>(tbase);
}

}  // namespace adaspark
