// K3 on the int8 tensor cores: cube scores of Eq. 1 from error-free digit slices.
//
// The selection must follow an fp64 evaluation of Eqs. 1-2 (rows may differ only inside a 1e-6
// probability margin), so plain bf16/fp32 tensor-core arithmetic is not accurate enough.  Instead
// every query row q and every mean key k are written in fixed point relative to the largest
// exponent of their row,
//     x = 2^(e - 29) * (d0*2^24 + d1*2^16 + d2*2^8 + d3),   digits d_i signed bytes in [-128, 127],
// (exact for elements within 2^-22 (q, 8 significant bits) / 2^-6 (k, 24 bits) of the row maximum,
// rounded at 2^-29 of it below that).  tcgen05.mma of kind::i8 multiplies the digit planes with exact
// int32 accumulation:  S_L = sum_{a+b=L} Q_a . K_b  for each level L (|S_L| <= 4 * 128 * 2^14).  Then
//     q . k = 2^(e_q + e_k - 10) * (S_0 + S_1*2^-8 + S_2*2^-16 + S_3*2^-24 + levels >= 4),
// and the levels 0..3 (10 digit pairs, four TMEM accumulators) are combined exactly in fp64.  The
// dropped levels are bounded by about 5e-7 in the scaled logit for |q| <= 3, |k| <= 5 in the worst
// case (all digit products aligned) and typically 10x less: inside the margin above.  A digit plane
// row is always 128 bytes (head_dim 64 is zero-padded).
//
//   slice_keys_kernel   digit planes + row exponents of the mean keys (once per forward, tiny)
//   score_tc_kernel     persistent CTAs, one per SM; work item = one 128-row query tile x a group of
//                       64-cube column tiles.  Roles (576 threads), pipelined across items:
//     warps 0-7   epilogue (thread = row = TMEM lane, 32 of the 64 columns): TMEM -> fp64 scores ->
//                 coalesced rows of the score buffer.  The four level accumulators are double-buffered
//                 in TMEM (2 x 4 x 64 columns), so the epilogue of one column tile overlaps the MMAs of
//                 the next
//     warps 8-15  slicers (two threads per row): read the bf16 query row early, then write the four
//                 swizzled digit planes of the tile into shared memory once the previous item's MMAs
//                 have released them
//     warp 16     TMA producer: key digit blocks (one plane of 64 cubes, 8 KB) in a ring
//     warp 17     issues the tcgen05.mma stream (40 of 128x64x32 per column tile)
#pragma once
#include "tc_common.cuh"

namespace adaspark {

constexpr int kScoreTcThreads = 576;
constexpr int kScoreTcRing = 8;          // key digit blocks (64 cubes x 128 bytes, 8 KB) in flight
constexpr int kScoreTcCols = 64;         // cubes per column tile
constexpr int kDigitRowBytes = 128;      // bytes per row of a digit plane

// The four signed base-256 digits of v = round(x * 2^(29 - e)) (|v| < 2^30), packed in one word:
// byte 3 = d0 (most significant) ... byte 0 = d3.  Adding 0x80 to every byte position turns the
// balanced digits into the plain unsigned bytes of v + 0x80808080, so two integer operations give
// all four.
__device__ __forceinline__ uint32_t packed_digits(float x, float mult) {
    const uint32_t u = (uint32_t)__float2int_rn(x * mult) + 0x80808080u;
    return u ^ 0x80808080u;
}
__device__ __forceinline__ float digit_scale(int e) {             // 2^(29 - e), exact for e >= -97
    return __int_as_float((156 - e) << 23);
}
__device__ __forceinline__ int row_exponent_from_field(int biased) {   // 8-bit exponent field of the row maximum
    return biased == 0 ? 0 : max(biased - 127, -90);               // rows smaller than 2^-90 keep fewer digits
}
// Byte k of four packed words -> one word (element i in byte i): digit plane 3 - k of four elements.
template <int k>
__device__ __forceinline__ uint32_t gather_byte(uint32_t w0, uint32_t w1, uint32_t w2, uint32_t w3) {
    const uint32_t lo = __byte_perm(w0, w1, (uint32_t)k | ((uint32_t)(4 + k) << 4));
    const uint32_t hi = __byte_perm(w2, w3, (uint32_t)k | ((uint32_t)(4 + k) << 4));
    return __byte_perm(lo, hi, 0x5410);
}

// Digit planes of the mean keys: planes[p][(b*Hkv+gk)*N_ld + cube][128 bytes] (int8, zero beyond D),
// key_exp[(b*Hkv+gk)*N_ld + cube].  One warp per cube row, four elements per lane; rows >= N inside
// the padded leading dimension are zero-filled.
__global__ void __launch_bounds__(128) slice_keys_kernel(Geom g, const float* __restrict__ cube_keys,
                                                         unsigned char* __restrict__ planes, int32_t* __restrict__ key_exp) {
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5);              // (b*Hkv+gk)*N_ld + cube
    const int n_rows = g.B * g.Hkv * g.N_ld;
    if (row >= n_rows) return;
    const int bh = row / g.N_ld, cube = row - bh * g.N_ld;
    const size_t plane_stride = (size_t)n_rows * kDigitRowBytes;
    const bool live = cube < g.N && lane * 4 < g.D;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (live) x = *reinterpret_cast<const float4*>(cube_keys + ((size_t)bh * g.N + cube) * g.D + lane * 4);
    float mx = fmaxf(fmaxf(fabsf(x.x), fabsf(x.y)), fmaxf(fabsf(x.z), fabsf(x.w)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const int e = row_exponent_from_field((int)((__float_as_uint(mx) >> 23) & 0xffu));
    const float mult = digit_scale(e);
    const uint32_t w0 = packed_digits(x.x, mult), w1 = packed_digits(x.y, mult);
    const uint32_t w2 = packed_digits(x.z, mult), w3 = packed_digits(x.w, mult);
    unsigned char* dst = planes + (size_t)row * kDigitRowBytes + lane * 4;
    *reinterpret_cast<uint32_t*>(dst) = gather_byte<3>(w0, w1, w2, w3);
    *reinterpret_cast<uint32_t*>(dst + plane_stride) = gather_byte<2>(w0, w1, w2, w3);
    *reinterpret_cast<uint32_t*>(dst + 2 * plane_stride) = gather_byte<1>(w0, w1, w2, w3);
    *reinterpret_cast<uint32_t*>(dst + 3 * plane_stride) = gather_byte<0>(w0, w1, w2, w3);
    if (lane == 0) key_exp[row] = e;
}

template <int D>
struct ScoreTcSmem {
    unsigned char qd[4][128][kDigitRowBytes];           // digit planes of the Q tile, UMMA layout (128-B swizzle)
    unsigned char kring[kScoreTcRing][kScoreTcCols][kDigitRowBytes];   // key digit blocks: one plane of 64 cubes
    double stage[2][128][32];                           // epilogue, per column half: scores of 32 columns, index ^ (row & 31)
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
    constexpr int kBlocks = 4;                                    // key digit blocks (planes) per column tile
    constexpr uint32_t kIdesc = tc::make_idesc_s8(128, kScoreTcCols);
    constexpr uint32_t kBlockBytes = kScoreTcCols * kDigitRowBytes;
    constexpr int kProducerWarp = 16, kMmaWarp = 17;

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
            tc::mbar_init(&sm.acc_free[i], 256);
        }
        sm.abort_flag = 0;
        tc::fence_barrier_init();
    }
    if (D < kDigitRowBytes) {                                     // bytes beyond head_dim stay zero for the whole kernel
        uint4* z = reinterpret_cast<uint4*>(&sm.qd[0][0][0]);
        for (int i = tid; i < (int)(sizeof(sm.qd) / 16); i += kScoreTcThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
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
                        const int plane = blk, s = i % kScoreTcRing, u = i / kScoreTcRing;
                        if (blk == 0 && !(ok = tc::mbar_wait(&sm.k_group_empty[s >> 2], (u & 1) ^ 1, abort_flag))) break;
                        tc::mbar_arrive_expect_tx(&sm.k_full[s], kBlockBytes);
                        tc::tma_load_2d(&sm.kring[s][0][0], &tmK, 0, plane * n_rows + k_row0 + ct * kScoreTcCols, &sm.k_full[s]);
                    }
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t kPlaneStep = (uint32_t)sizeof(sm.qd[0]) >> 4;
            constexpr uint32_t kRingStep = (uint32_t)sizeof(sm.kring[0]) >> 4, kKStep = 32 >> 4;
            const uint32_t q_lo0 = tc::smem_desc_lo_sw128(smem_u32(&sm.qd[0][0][0]));
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
                    // fully unrolled: every descriptor is a base plus a compile-time offset
#pragma unroll
                    for (int blk = 0; blk < kBlocks; ++blk) {
                        const int s = i % kScoreTcRing, u = i / kScoreTcRing;
                        ++i;
                        if (ok && !(ok = tc::mbar_wait(&sm.k_full[s], u & 1, abort_flag))) break;
                        tc::tc_fence_after_sync();
                        const uint32_t kb = k_lo0 + s * kRingStep;
#pragma unroll
                        for (int a = 0; a + blk <= 3; ++a) {      // plane blk of the keys, plane a of the queries: level a + blk
                            const uint32_t qa = q_lo0 + a * kPlaneStep;
                            const uint32_t dst = tbase + buf * 256 + (a + blk) * kScoreTcCols;
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)
                                tc::umma_ss_i8(dst, tc::smem_desc_from_halves(qa + ks * kKStep, tc::kSmemDescHiSw128),
                                               tc::smem_desc_from_halves(kb + ks * kKStep, tc::kSmemDescHiSw128), kIdesc,
                                               !(blk == 0 && ks == 0));
                        }
                        if (blk == 3) tc::umma_commit(&sm.k_group_empty[s >> 2]);
                    }
                    if (ok) tc::umma_commit(&sm.acc_full[buf]);
                }
                if (ok) tc::umma_commit(&sm.qd_free);             // the digit planes may be overwritten
                ++n_done;
            }
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------ slicers (two threads per row)
        constexpr int kChunks = D / 16;                           // 16-byte chunks (8 elements) of the row half
        constexpr int kOut = D / 32;                              // 16-byte chunks (16 digits) per plane per thread
        const int r = (tid - 256) >> 1, half = (tid - 256) & 1;
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
            const float mult = digit_scale(row_exponent_from_field((int)(mxbits >> 7)));
            // the previous item's MMAs must have finished reading the digit planes
            if (n_done > 0 && !(ok = tc::mbar_wait(&sm.qd_free, (n_done - 1) & 1, abort_flag))) break;
            unsigned char* dst = &sm.qd[0][0][0];
#pragma unroll
            for (int o = 0; o < kOut; ++o) {
                uint32_t pw[4][4];                                // [plane][4 elements per word]
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {                  // elements 16*o + 4*q4 .. +3 = two packed bf16 words
                    const uint4 vv = v[2 * o + (q4 >> 1)];
                    const uint32_t wa = (q4 & 1) ? vv.z : vv.x, wb = (q4 & 1) ? vv.w : vv.y;
                    const uint32_t w0 = packed_digits(__uint_as_float(wa << 16), mult);
                    const uint32_t w1 = packed_digits(__uint_as_float(wa & 0xffff0000u), mult);
                    const uint32_t w2 = packed_digits(__uint_as_float(wb << 16), mult);
                    const uint32_t w3 = packed_digits(__uint_as_float(wb & 0xffff0000u), mult);
                    pw[0][q4] = gather_byte<3>(w0, w1, w2, w3);
                    pw[1][q4] = gather_byte<2>(w0, w1, w2, w3);
                    pw[2][q4] = gather_byte<1>(w0, w1, w2, w3);
                    pw[3][q4] = gather_byte<0>(w0, w1, w2, w3);
                }
                const int off = sw128(r, half * kOut + o);        // 16-byte chunk of the 128-byte plane row
#pragma unroll
                for (int pl = 0; pl < 4; ++pl)
                    *reinterpret_cast<uint4*>(dst + (size_t)pl * sizeof(sm.qd[0]) + off) = make_uint4(pw[pl][0], pw[pl][1], pw[pl][2], pw[pl][3]);
            }
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // digit planes visible to the tensor core
            tc::mbar_arrive(&sm.q_sliced);
            ++n_done;
        }
    } else {
        // ------------------------------------------------------------ epilogue (thread = row = TMEM lane)
        const int lg = warp & 3, chalf = warp >> 2;               // TMEM lane group, column half of the tile
        const int r = lg * 32 + lane;
        const uint32_t lane_addr = tbase + ((uint32_t)(lg * 32) << 16);
        double (*stage)[32] = sm.stage[chalf];
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
                e_q = row_exponent_from_field((int)(mxbits >> 7));
            }
            const double rowf = __hiloint2double((1023 + e_q) << 20, 0);          // 2^e_q
            const int32_t* kexp = key_exp + (size_t)(w.b * g.Hkv + w.gk) * g.N_ld;
            double* out_rows = logits + (size_t)w.tile_in_chunk * kTileRows * g.N_ld;
            for (int ct = w.ct0; ok && ct < w.ct1; ++ct, ++c_run) {
                const int buf = c_run & 1;
                if (!(ok = tc::mbar_wait(&sm.acc_full[buf], (c_run >> 1) & 1, abort_flag))) break;
                tc::tc_fence_after_sync();
                {
                    const int col0 = ct * kScoreTcCols + chalf * 32;   // this warp's 32 columns
                    // column factor 2^(e_k - 34) * scale, held by the lane that owns the column
                    const int jc = col0 + lane;
                    const int ek = jc < g.N_ld ? kexp[jc] : 0;
                    const double colf = __hiloint2double((1023 + ek - 34) << 20, 0) * g.scale_d;
#pragma unroll
                    for (int hc = 0; hc < 2; ++hc) {
                        uint32_t lv[4][16];
#pragma unroll
                        for (int L = 0; L < 4; ++L) tc::tmem_ld_32x16(lane_addr + buf * 256 + L * kScoreTcCols + chalf * 32 + hc * 16, lv[L]);
                        tc::tmem_wait_ld();
                        if (hc == 1) {                            // last read of this accumulator set: release it
                            tc::tc_fence_before_sync();
                            tc::mbar_arrive(&sm.acc_free[buf]);
                        }
#pragma unroll
                        for (int i = 0; i < 16; ++i) {
                            // exact integer level sums: S0*2^24 + S1*2^16 + S2*2^8 + S3 = hi*2^16 + lo
                            const int hi = (int)lv[0][i] * 256 + (int)lv[1][i];
                            const int lo = (int)lv[2][i] * 256 + (int)lv[3][i];
                            const double hd = __hiloint2double(0x43300000, hi ^ 0x80000000) - 4503601774854144.0;   // (double)hi
                            const double ld = __hiloint2double(0x43300000, lo ^ 0x80000000) - 4503601774854144.0;   // 2^52 + 2^31
                            const double v = fma(hd, 65536.0, ld);
                            const int col = hc * 16 + i;
                            const double cf = __shfl_sync(0xffffffffu, colf, col);
                            stage[r][col ^ (r & 31)] = (v * rowf) * cf;
                        }
                    }
                    __syncwarp();
                    if (col0 + lane < g.N_ld) {
                        for (int rr = 0; rr < 32; ++rr) {
                            const int row = lg * 32 + rr;
                            out_rows[(size_t)row * g.N_ld + col0 + lane] = stage[row][lane ^ (row & 31)];
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
