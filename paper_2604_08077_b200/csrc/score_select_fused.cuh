// K3: cube scoring (Eq. 1) and nucleus selection (Eq. 2) in ONE kernel; no score ever leaves the SM.
//
// Scores.  The selection must follow an fp64 evaluation of Eqs. 1-2 (rows may differ only inside a
// 1e-6 probability margin), so plain bf16/fp32 tensor-core arithmetic is not accurate enough.  Every
// query row q and every mean key k are written in fixed point,
//     x = 2^(e - 29) * (d0*2^24 + d1*2^16 + d2*2^8 + d3),   digits d_i signed bytes in [-128, 127],
// with e the exponent of the largest element of the query row (e_q) or of all mean keys of the
// (batch, kv head) (E_K).  tcgen05.mma of kind::i8 multiplies the digit planes with exact int32
// accumulation,  S_L = sum_{a+b=L} Q_a . K_b  (10 digit pairs, levels L = 0..3, four TMEM
// accumulators), and
//     q . k_j = 2^(e_q + E_K - 34) * V_j,      V_j = S_0*2^24 + S_1*2^16 + S_2*2^8 + S_3   (an int64),
// up to the dropped levels >= 4 and the rounding of elements far below the row maximum.  Because the
// key exponent is shared by the whole head, all scores of a row are the SAME positive factor
// f = 2^(e_q + E_K - 34) * scale times an integer: order and distances between the scores of a row
// are integer arithmetic.  Rows whose exponents are so large that the fixed-point error could reach
// the margin (f > kMaxScorePerUnit) are not decided here: they go to the fp64 kernel of
// select_exact.cuh through a list in the workspace, and so does any row this kernel gives up on.
//
// Selection (query row = TMEM lane).  The scores of a
// 128-row tile are far too many to keep (128 x up to 4096), and the tensor pipe is nearly idle, so
// the kernel RECOMPUTES them: it makes several passes over the tile's column tiles (64 cubes each),
// re-issuing the same MMAs, and each row narrows a key interval that holds its nucleus boundary:
//   pass A   (3 digit pairs only) the largest V_hi = S_0*256 + S_1 of the row gives an anchor
//            V_A >= max_j V_j;  the order key of cube j is  delta_j = V_A - V_j >= 0  (smaller first)
//   pass 0   histogram of the fixed-point masses m_j = round(2^38 * exp(-delta_j * f)) over 64
//            buckets of delta >> sh (bucket 63 catches everything beyond); Z = sum m_j,
//            T = ceil(p * Z); the bucket in which the cumulative mass crosses T holds the boundary
//   pass k   while that bucket holds more than kCandCap cubes: the same over 64 sub-buckets of it
//   last     cubes above the interval are selected (bits written), those inside are collected
//            (at most kCandCap) and the crossing cube is found among them directly.
// Rows of a tile advance independently; the tile makes passes until every row is done (at least two,
// so that the MMA stream never waits for the decision).  Masses are integers, so sums do not depend
// on their order; a mass is quantised to 2^-38 of the row maximum, which moves no cumulative
// probability by more than n * 2^-39.  Equal scores are ordered by lower cube index.
// Top-K (top_k > 0): the same with every mass = 1 and T = min(top_k, candidates).
//
// A row is served by FOUR threads (same TMEM lane, four warps): each takes 16 of the 64 columns of every
// column tile, adds to the row's histogram with shared-memory atomics and appends to the row's candidate
// list through an atomic counter; what the four must agree on (anchor, crossing bucket, boundary key)
// goes through small shared arrays between barriers of the 512 selection threads.  The work of a row is
// latency-bound (TMEM loads, fp64 chains, shared-memory atomics), so four warps per scheduler matter
// more than instruction count: with one thread per row the MMA thread waited 3/4 of the time.
//
// Roles (768 threads, one persistent CTA per SM, work item = one 128-row query tile, long tiles first):
//   warps 0-15   selection: warp w serves TMEM lane quarter w % 4 (rows 32*(w%4) + lane) and columns
//                16*(w/4) .. +15 of every column tile.  An accumulator set is freed as soon as its values
//                are in registers
//   warps 16-19  slicers (one thread per row): digit planes of the next tile's queries into shared memory
//   warp 20      TMA producer: key digit planes of one column tile (4 x 8 KB; 2 x 8 KB in pass A), 2 slots
//   warps 21-22  issue the tcgen05.mma stream (40 of 128x64x32 per column tile, 12 in pass A; half each)
//                into double-buffered accumulator sets (2 x 4 levels x 64 columns = all 512 TMEM columns);
//                each warp runs converged and issues through one elected lane
//   warp 23      idle (it completes the sixth warpgroup for the register re-allocation)
#pragma once
#include "tc_common.cuh"

namespace adaspark {

constexpr int kFusedThreads = 768;
constexpr int kSelThreads = 512;         // selection threads: four per row
constexpr int kScoreTcCols = 64;         // cubes per column tile
constexpr int kDigitRowBytes = 128;      // bytes per row of a digit plane
constexpr int kCandCap = 24;             // cubes a row may collect from its boundary interval
constexpr int kMaxHistPasses = 10;       // histogram passes a row may take before it is handed to the fp64 kernel
// Largest score per unit of V (f) this kernel decides itself: 2^(6 - 34) / sqrt(64), i.e. exponents up to
// e_q + E_K = 6 at the default scale of head_dim 64 (the fixed-point error grows with f; the benchmark
// inputs reach e_q + E_K = 5 at head_dim 128)
constexpr double kMaxScorePerUnit = 0.125 / 268435456.0;
// Per-thread registers after setmaxnreg.  The re-allocation only moves registers inside the CTA's launch
// allocation (768 threads x 80): 4 * 88 + 88 + 40 = 6 * 80.  (A sum above it would block forever.)
constexpr int kSelRegs = 88, kSlicerRegs = 88, kIssueRegs = 40;
static_assert(4 * kSelRegs + kSlicerRegs + kIssueRegs <= 6 * 80, "setmaxnreg budget exceeds the launch allocation");

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

// Largest |mean key element| of every (batch, kv head), as float bits (non-negative floats order like
// their bit patterns): head_max_bits[b*Hkv + gk], zeroed by the caller.  grid (B*Hkv, 8).
__global__ void __launch_bounds__(256) key_exponent_kernel(Geom g, const float* __restrict__ cube_keys,
                                                           uint32_t* __restrict__ head_max_bits) {
    const int bh = blockIdx.x;
    const size_t n4 = (size_t)g.N_live * g.D / 4;             // the cubes present so far
    const float4* src = reinterpret_cast<const float4*>(cube_keys + (size_t)bh * g.N * g.D);
    uint32_t mx = 0;
    for (size_t i = (size_t)blockIdx.y * 256 + threadIdx.x; i < n4; i += (size_t)gridDim.y * 256) {
        const float4 x = src[i];
        mx = max(max(mx, __float_as_uint(fabsf(x.x))), max(__float_as_uint(fabsf(x.y)),
                 max(__float_as_uint(fabsf(x.z)), __float_as_uint(fabsf(x.w)))));
    }
    mx = __reduce_max_sync(0xffffffffu, mx);
    if ((threadIdx.x & 31) == 0 && mx) atomicMax(head_max_bits + bh, mx);
}
__device__ __forceinline__ int head_exponent(uint32_t max_bits) { return row_exponent_from_field((int)((max_bits >> 23) & 0xffu)); }

// Digit planes of the mean keys: planes[p][(b*Hkv+gk)*N_ld + cube][128 bytes] (int8, zero beyond D), all
// cubes of a (batch, kv head) in the fixed point of that head's exponent.  One warp per cube row, four
// elements per lane; rows >= N inside the padded leading dimension are zero-filled.
__global__ void __launch_bounds__(128) slice_keys_kernel(Geom g, const float* __restrict__ cube_keys,
                                                         const uint32_t* __restrict__ head_max_bits,
                                                         unsigned char* __restrict__ planes) {
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5);              // (b*Hkv+gk)*N_ld + cube
    const int n_rows = g.B * g.Hkv * g.N_ld;
    if (row >= n_rows) return;
    const int bh = row / g.N_ld, cube = row - bh * g.N_ld;
    const size_t plane_stride = (size_t)n_rows * kDigitRowBytes;
    const bool live = cube < g.N_live && lane * 4 < g.D;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (live) x = *reinterpret_cast<const float4*>(cube_keys + ((size_t)bh * g.N + cube) * g.D + lane * 4);
    const float mult = digit_scale(head_exponent(head_max_bits[bh]));
    const uint32_t w0 = packed_digits(x.x, mult), w1 = packed_digits(x.y, mult);
    const uint32_t w2 = packed_digits(x.z, mult), w3 = packed_digits(x.w, mult);
    unsigned char* dst = planes + (size_t)row * kDigitRowBytes + lane * 4;
    *reinterpret_cast<uint32_t*>(dst) = gather_byte<3>(w0, w1, w2, w3);
    *reinterpret_cast<uint32_t*>(dst + plane_stride) = gather_byte<2>(w0, w1, w2, w3);
    *reinterpret_cast<uint32_t*>(dst + 2 * plane_stride) = gather_byte<1>(w0, w1, w2, w3);
    *reinterpret_cast<uint32_t*>(dst + 3 * plane_stride) = gather_byte<0>(w0, w1, w2, w3);
}

// round(2^38 * exp(x)) for x <= 0 as an integer (0 below about -27): argument reduction by ln 2,
// degree-10 Taylor polynomial on |r| <= 0.347 (relative error < 1e-12), the exponent spliced in as
// an integer, then one magic-number addition rounds to the nearest integer.
__device__ __forceinline__ unsigned long long mass38(double x) {
    x = fmax(x, -64.0);
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
    const double scaled = __hiloint2double(__double2hiint(p) + ((k + 38) << 20), __double2loint(p));   // p * 2^(k+38)
    const double v = scaled + 4503599627370496.0;                       // 2^52 + round(scaled)
    return (unsigned long long)__double_as_longlong(v) & 0xFFFFFFFFFFFFFull;
}

template <int D>
struct FusedSmem {
    unsigned char qd[4][128][kDigitRowBytes];                      // digit planes of the Q tile, UMMA layout (128-B swizzle)
    unsigned char kring[2][4][kScoreTcCols][kDigitRowBytes];       // key digit planes of a column tile, two slots
    unsigned long long hist[64][128];                              // [bucket][row]: (sum of masses << 13) | count
    unsigned long long cand[kCandCap][128];                        // [slot][row]: (delta << 12) | cube
    unsigned long long part[4][128];                               // what the four threads of a row exchange
    unsigned long long res_base[128];                              // crossing bucket of a row: mass before it ...
    int32_t res_cb[128];                                           // ... and bucket | count << 8
    int32_t cand_cnt[128];                                         // candidates appended by the row's threads
    int32_t row_count[128];                                        // |S_i| of the row
    uint32_t tile_union[2][128];                                   // OR over the tile's rows of each selection word
    int32_t eq[2][128];                                            // exponent e_q of each row of the tile (by tile parity)
    int32_t need[4];                                               // decision ring: d + 1 = "another pass after the next"
    uint64_t q_sliced, qd_free, k_full[2], acc_full[2], acc_free[2], decided[4], sel_sync, quarter_sync[4];
    uint32_t tmem_base;
    int abort_flag;
};

// Work item `it` of the launch: long (late) tiles first.
struct FusedItem {
    int b, h, gk, tile, n_ct;
};
__device__ __forceinline__ FusedItem fused_item(const Geom& g, int it) {
    FusedItem w;
    const int n_hb = g.B * g.Hq;
    const int lvl = it / n_hb, hb = it - lvl * n_hb;
    w.tile = g.n_tiles - 1 - lvl;
    g.div_Hq.divmod(hb, w.b, w.h);
    w.gk = w.h / g.G;
    w.n_ct = (tile_max_candidates(g, w.tile) + kScoreTcCols - 1) / kScoreTcCols;
    return w;
}

__device__ __forceinline__ void tmem_ld_32x8(uint32_t taddr, uint32_t (&r)[8]) {   // 8 consecutive columns
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "r"(taddr)
                 : "memory");
}

__device__ __forceinline__ void tmem_ld_32x4(uint32_t taddr, uint32_t* r) {   // 4 consecutive columns
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(taddr)
                 : "memory");
}

// q: the call's queries [B, S_io, Hq, D].  tile_mask as mask_index() describes;
// tile_union[((b*Hq+h)*n_tiles_cap + tile)*n_words + w] = OR of word w over the tile's rows.
// fallback_rows[0 .. *fallback_count) receives ((b*Hq+h)*n_tiles_cap + tile)*128 + r of the rows left
// to the fp64 kernel.
template <int D, bool kByCount>
__global__ void __launch_bounds__(kFusedThreads, 1) score_select_fused_kernel(
    Geom g, int n_items, const __nv_bfloat16* __restrict__ q, const __grid_constant__ CUtensorMap tmK,
    const uint32_t* __restrict__ head_max_bits, uint32_t* __restrict__ tile_mask, uint32_t* __restrict__ tile_union,
    uint32_t* __restrict__ sel_bitmap, int32_t* __restrict__ sel_count, int32_t* __restrict__ fallback_rows,
    uint32_t* __restrict__ fallback_count, int32_t* __restrict__ status) {
    extern __shared__ unsigned char fused_raw[];
    FusedSmem<D>& sm = *reinterpret_cast<FusedSmem<D>*>((reinterpret_cast<uintptr_t>(fused_raw) + 1023) & ~(uintptr_t)1023);
    constexpr uint32_t kIdesc = tc::make_idesc_s8(128, kScoreTcCols);
    constexpr uint32_t kPlaneBytes = kScoreTcCols * kDigitRowBytes;
    constexpr int kSlicerWarp0 = 16, kProducerWarp = 20, kMmaWarp = 21;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0) {
        tc::mbar_init(&sm.q_sliced, 4);                     // one arrival per slicer warp
        tc::mbar_init(&sm.qd_free, 2);
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(&sm.k_full[i], 1);
            tc::mbar_init(&sm.acc_full[i], 2);                // one commit per MMA-issuing thread
            tc::mbar_init(&sm.acc_free[i], kSelThreads / 32);   // one arrival per selection warp:
            // 512 single arrivals on one barrier word serialise and cost more than the work between them
        }
        for (int i = 0; i < 4; ++i) {
            tc::mbar_init(&sm.decided[i], kSelThreads / 32);
            sm.need[i] = 0;
        }
        tc::mbar_init(&sm.sel_sync, kSelThreads / 32);
        for (int i = 0; i < 4; ++i) tc::mbar_init(&sm.quarter_sync[i], 4);   // the four warps that share 32 rows
        sm.abort_flag = 0;
        tc::fence_barrier_init();
    }
    // selection state that must start at zero
    for (int i = tid; i < 64 * 128; i += kFusedThreads) (&sm.hist[0][0])[i] = 0ull;
    if (tid < 128) { sm.cand_cnt[tid] = 0; sm.row_count[tid] = 0; sm.tile_union[0][tid] = 0u; sm.tile_union[1][tid] = 0u; }
    if (D < kDigitRowBytes) {                                     // bytes beyond head_dim stay zero for the whole kernel
        uint4* z = reinterpret_cast<uint4*>(&sm.qd[0][0][0]);
        for (int i = tid; i < (int)(sizeof(sm.qd) / 16); i += kFusedThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
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

    // Does the tile make histogram/collect pass f (f >= 2)?  Decision d = d0 + f - 2 was published by the
    // selection warps after pass f - 2.  Every role evaluates this with the same arguments, so all of
    // them walk the same sequence of jobs.
    auto another_pass = [&](int d, bool& ok) -> bool {
        ok = tc::mbar_wait(&sm.decided[d & 3], (d >> 2) & 1, abort_flag);
        return ok && *reinterpret_cast<volatile int32_t*>(&sm.need[d & 3]) == d + 1;
    };

    if (warp >= kProducerWarp) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kIssueRegs));
    }

    if (warp == kProducerWarp) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const int n_rows = g.B * g.Hkv * g.N_ld;
            int c = 0, d0 = 0;                                    // running job / decision counters of this CTA
            bool ok = true;
            for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x) {
                const FusedItem w = fused_item(g, it);
                if (w.n_ct == 0) continue;
                const int k_row0 = (w.b * g.Hkv + w.gk) * g.N_ld;
                int f = -1;                                       // -1: anchor pass, then passes 0, 1, ...
                while (ok) {
                    const int n_planes = f < 0 ? 2 : 4;
                    for (int ct = 0; ok && ct < w.n_ct; ++ct, ++c) {
                        const int s = c & 1, use = c >> 1;
                        if (use > 0 && !(ok = tc::mbar_wait(&sm.acc_full[s], (use - 1) & 1, abort_flag))) break;   // the slot's last reader has finished
                        tc::mbar_arrive_expect_tx(&sm.k_full[s], n_planes * kPlaneBytes);
                        for (int pl = 0; pl < n_planes; ++pl)
                            tc::tma_load_2d(&sm.kring[s][pl][0][0], &tmK, 0, pl * n_rows + k_row0 + ct * kScoreTcCols, &sm.k_full[s]);
                    }
                    ++f;
                    if (f >= 2 && !another_pass(d0 + f - 2, ok)) break;
                }
                d0 += f;
            }
        }
    } else if (warp == kMmaWarp || warp == kMmaWarp + 1) {
        // ------------------------------------------------------------ MMA issuers
        // Two threads issue the stream (one thread gets a 128x64x32 MMA accepted every ~90 - 110 cycles, the
        // tensor core would take them faster): issuer 0 owns the accumulators of levels 0 and 3, issuer 1 those
        // of levels 1 and 2 (five digit pairs each, no accumulator shared); a job is ready when both have
        // committed.  (Three issuers, 16 / 12 / 12 MMAs per column tile, measured 0.7 % slower.)
        const int issuer = warp - kMmaWarp;
        {
            // The whole warp walks the jobs and one elected lane issues, with every operand warp-uniform: a thread
            // gets its MMAs accepted faster that way than from a branch that lane 0 alone enters.
            constexpr uint32_t kQPlaneStep = (uint32_t)sizeof(sm.qd[0]) >> 4, kKPlaneStep = (uint32_t)sizeof(sm.kring[0][0]) >> 4;
            constexpr uint32_t kSlotStep = (uint32_t)sizeof(sm.kring[0]) >> 4, kKStep = 32 >> 4;
            const uint32_t q_lo0 = __shfl_sync(0xffffffffu, tc::smem_desc_lo_sw128(smem_u32(&sm.qd[0][0][0])), 0);
            const uint32_t k_lo0 = __shfl_sync(0xffffffffu, tc::smem_desc_lo_sw128(smem_u32(&sm.kring[0][0][0][0])), 0);
            const uint32_t tb = __shfl_sync(0xffffffffu, tbase, 0);
            bool ok = true;
            int c = 0, d0 = 0, n_done = 0;
            for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x) {
                const FusedItem w = fused_item(g, it);
                if (w.n_ct == 0) continue;
                if (!(ok = tc::mbar_wait_warp(&sm.q_sliced, n_done & 1, abort_flag))) break;
                int f = -1;
                while (ok) {
                    for (int ct = 0; ok && ct < w.n_ct; ++ct, ++c) {
                        const int s = c & 1, use = c >> 1;
                        if (use > 0 && !(ok = tc::mbar_wait_warp(&sm.acc_free[s], (use - 1) & 1, abort_flag))) break;
                        if (!(ok = tc::mbar_wait_warp(&sm.k_full[s], use & 1, abort_flag))) break;
                        tc::tc_fence_after_sync();
                        const uint32_t kb0 = k_lo0 + s * kSlotStep;
                        // level L = a + blk: plane a of the queries, plane blk of the keys; the anchor pass
                        // computes levels 0 and 1 only (S_0 = Q_0 K_0, S_1 = Q_0 K_1 + Q_1 K_0)
                        const int n_levels = f < 0 ? 2 : 4;
                        if (tc::elect_one()) {
#pragma unroll
                            for (int L = 0; L < 4; ++L) {
                                if (L >= n_levels || ((L == 0 || L == 3) ? 0 : 1) != issuer) continue;
#pragma unroll
                                for (int a = 0; a <= L; ++a)
#pragma unroll
                                    for (int ks = 0; ks < 4; ++ks)
                                        tc::umma_ss_i8(tb + s * 256 + L * kScoreTcCols,
                                                       tc::smem_desc_from_halves(q_lo0 + a * kQPlaneStep + ks * kKStep, tc::kSmemDescHiSw128),
                                                       tc::smem_desc_from_halves(kb0 + (L - a) * kKPlaneStep + ks * kKStep, tc::kSmemDescHiSw128),
                                                       kIdesc, !(a == 0 && ks == 0));
                            }
                            tc::umma_commit(&sm.acc_full[s]);         // accumulators ready; the key slot may be reloaded
                        }
                        __syncwarp();
                    }
                    ++f;
                    if (f >= 2) {
                        const bool more = __all_sync(0xffffffffu, another_pass(d0 + f - 2, ok));
                        ok = __all_sync(0xffffffffu, ok);
                        if (!more) break;
                    }
                }
                d0 += f;
                if (ok && tc::elect_one()) tc::umma_commit(&sm.qd_free);   // the digit planes may be overwritten (both issuers)
                __syncwarp();
                ++n_done;
            }
        }
    } else if (warp >= kSlicerWarp0 && warp < kProducerWarp) {
        // ------------------------------------------------------------ slicers (one thread per row)
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kSlicerRegs));
        const int r = tid - kSlicerWarp0 * 32;
        bool ok = true;
        int n_done = 0;
        for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x) {
            const FusedItem w = fused_item(g, it);
            if (w.n_ct == 0) continue;
            const int pos = w.tile * kTileRows + r;
            const bool live = slot_live(g, pos);
            // the row is read where the caller left it (sequence order): no cube-major copy of Q exists
            const uint4* src = reinterpret_cast<const uint4*>(q + (live ? (io_row(g, w.b, pos) * g.Hq + w.h) * D : 0));
            // first sweep over the row (before the planes are free): its largest exponent
            uint32_t mxbits = 0;
            if (live) {
#pragma unroll
                for (int c = 0; c < D / 8; ++c) {
                    const uint4 v = __ldg(src + c);
                    const uint32_t wd[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) mxbits = max(mxbits, max(wd[i] & 0x7fffu, (wd[i] >> 16) & 0x7fffu));
                }
            }
            const int e_q = row_exponent_from_field((int)(mxbits >> 7));
            const float mult = digit_scale(e_q);
            // the previous tile's MMAs must have finished reading the digit planes (and its selection
            // threads are past reading their exponents of the tile before that)
            if (n_done > 0 && !(ok = tc::mbar_wait(&sm.qd_free, (n_done - 1) & 1, abort_flag))) break;
            sm.eq[n_done & 1][r] = e_q;
            unsigned char* dst = &sm.qd[0][0][0];
#pragma unroll 2
            for (int o = 0; o < D / 16; ++o) {                    // 16 elements = one 16-byte chunk of every plane
                const uint4 va = live ? __ldg(src + 2 * o) : make_uint4(0u, 0u, 0u, 0u);
                const uint4 vb = live ? __ldg(src + 2 * o + 1) : make_uint4(0u, 0u, 0u, 0u);
                uint32_t pw[4][4];                                // [plane][4 elements per word]
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {                  // elements 16*o + 4*q4 .. +3 = two packed bf16 words
                    const uint4 vv = (q4 >> 1) ? vb : va;
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
                const int off = sw128(r, o);                      // 16-byte chunk of the 128-byte plane row
#pragma unroll
                for (int pl = 0; pl < 4; ++pl)
                    *reinterpret_cast<uint4*>(dst + (size_t)pl * sizeof(sm.qd[0]) + off) = make_uint4(pw[pl][0], pw[pl][1], pw[pl][2], pw[pl][3]);
            }
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // digit planes visible to the tensor core
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&sm.q_sliced);
            ++n_done;
        }
    } else if (warp < kSlicerWarp0) {
        // ------------------------------------------------------------ selection (4 threads per row)
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kSelRegs));
        const int quarter = warp & 3, part = warp >> 2;
        const int r = quarter * 32 + lane;
        const uint32_t lane_addr = tbase + ((uint32_t)(quarter * 32) << 16);
        unsigned long long* hist = &sm.hist[0][r];                // bucket b at hist[b * 128]
        unsigned long long* cand = &sm.cand[0][r];                // slot k at cand[k * 128]
        enum { kDone = 0, kHist = 1, kCollect = 2 };
        constexpr long long kLoMax = 3ll * (1ll << 29) + (1ll << 23);      // >= |S_2*256 + S_3|
        constexpr unsigned long long kOpen = 1ull << 62;          // span of an interval without upper end
        bool ok = true;
        int c = 0, d0 = 0, n_done = 0, t_par = 0, n_sync = 0, n_qsync = 0;
        // barrier among the four warps that serve the same 32 rows (bounded like every other wait here)
        auto sync_rows = [&]() -> bool {
            __threadfence_block();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&sm.quarter_sync[quarter]);
            const bool done = tc::mbar_wait(&sm.quarter_sync[quarter], n_qsync & 1, abort_flag);
            ++n_qsync;
            return done;
        };
        // barrier among all 512 selection threads
        auto sync_selection = [&]() -> bool {
            __threadfence_block();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&sm.sel_sync);
            const bool done = tc::mbar_wait(&sm.sel_sync, n_sync & 1, abort_flag);
            ++n_sync;
            return done;
        };
        // this warp has read its part of accumulator set s (one arrival per warp)
        auto release_acc = [&](int s) {
            tc::tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&sm.acc_free[s]);
        };
        auto to_double = [](unsigned long long d) -> double {     // exact for d < 2^52
            return __hiloint2double(0x43300000 | (int)(d >> 32), (int)(uint32_t)d) - 4503599627370496.0;
        };
        for (int it = blockIdx.x; ok && it < n_items; it += gridDim.x, t_par ^= 1) {
            const FusedItem w = fused_item(g, it);
            const int pos = w.tile * kTileRows + r;
            const bool live = slot_live(g, pos);
            const int n = live ? n_candidates(g, pos) : 0;
            const int n_warp = __reduce_max_sync(0xffffffffu, n);
            const size_t gt_cap = (size_t)(w.b * g.Hq + w.h) * g.n_tiles_cap + w.tile;
            uint32_t* mask_row = tile_mask + gt_cap * g.n_words * kTileRows + r;        // word w at mask_row[w * 128]
            const bool extra = live && (sel_bitmap != nullptr || sel_count != nullptr);
            const size_t raster_row = extra ? (size_t)(w.b * g.Hq + w.h) * g.S_io + (pos_to_io(g, pos) - g.pos_begin) : 0;
            uint32_t* bm_row = (extra && sel_bitmap) ? sel_bitmap + raster_row * g.n_words : nullptr;
            // every word starts at zero: the collect pass ORs the selected cubes' bits into them
            for (int wd = part; wd < g.n_words; wd += 4) {
                mask_row[(size_t)wd * kTileRows] = 0u;
                if (bm_row) bm_row[wd] = 0u;
            }
            bool give_up = false;
            if (w.n_ct > 0) {
                // ---------------- anchor pass: largest S_0*256 + S_1 over the row's candidates
                int max_hi = INT_MIN;
                for (int ct = 0; ok && ct < w.n_ct; ++ct, ++c) {
                    const int s = c & 1;
                    if (!(ok = tc::mbar_wait(&sm.acc_full[s], (c >> 1) & 1, abort_flag))) break;
                    tc::tc_fence_after_sync();
                    const int col0 = ct * kScoreTcCols + part * 16;
                    if (col0 < n_warp) {
                        uint32_t l0[16], l1[16];
                        tc::tmem_ld_32x16(lane_addr + s * 256 + part * 16, l0);
                        tc::tmem_ld_32x16(lane_addr + s * 256 + kScoreTcCols + part * 16, l1);
                        tc::tmem_wait_ld();
                        release_acc(s);
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            if (col0 + i < n) max_hi = max(max_hi, (int)l0[i] * 256 + (int)l1[i]);
                    } else {
                        release_acc(s);
                    }
                }
                if (!ok) break;
                sm.part[part][r] = (unsigned long long)(long long)max_hi;
                if (!(ok = sync_rows())) break;
#pragma unroll
                for (int k = 0; k < 4; ++k) max_hi = max(max_hi, (int)(long long)sm.part[k][r]);
                // ---------------- per-row constants (the same in the row's four threads)
                const int e_sum = sm.eq[n_done & 1][r] + head_exponent(head_max_bits[w.b * g.Hkv + w.gk]);
                const double f = __hiloint2double((1023 + e_sum - 34) << 20, 0) * g.scale_d;   // score per unit of V
                const double neg_f = -f;
                const long long VA = (long long)max_hi * 65536 + kLoMax;   // anchor: >= every V_j of the row
                int sh = 0;                                       // first-level bucket width 2^sh * f in (1/8, 1/4]
                {
                    const int e = ((__double2hiint(0.25 / f) >> 20) & 0x7ff) - 1023;       // floor(log2(0.25 / f))
                    sh = min(max(e, 0), 50);
                }
                unsigned long long lo = 0ull, span = kOpen, base = 0ull, target = 0ull;
                int state = n > 0 ? kHist : kDone;
                bool first_level = true;
                if (n > 0 && !(f <= kMaxScorePerUnit)) { state = kDone; give_up = true; }   // also a non-finite f
                int hist_passes = 0;
                // ---------------- passes
                int fpass = 0;
                while (ok) {
                    const int my = state;                         // what this row does in this pass
                    const bool warp_idle = !__any_sync(0xffffffffu, my != kDone);
                    for (int ct = 0; ok && ct < w.n_ct; ++ct, ++c) {
                        const int s = c & 1;
                        if (!(ok = tc::mbar_wait(&sm.acc_full[s], (c >> 1) & 1, abort_flag))) break;
                        tc::tc_fence_after_sync();
                        // This thread's columns of the job: 4*part .. +3 of every group of 16 (interleaved, so
                        // that a ragged last column tile loads the row's four threads alike); half hf = one 32-cube word
#pragma unroll
                        for (int hf = 0; hf < 2; ++hf) {
                            const int colh = ct * kScoreTcCols + hf * 32 + part * 4;    // first column of this half
                            uint32_t bits = 0;
                            if (colh < n_warp && !warp_idle) {
                                uint32_t lv[4][8];
#pragma unroll
                                for (int L = 0; L < 4; ++L) {
                                    tmem_ld_32x4(lane_addr + s * 256 + L * kScoreTcCols + hf * 32 + part * 4, &lv[L][0]);
                                    tmem_ld_32x4(lane_addr + s * 256 + L * kScoreTcCols + hf * 32 + 16 + part * 4, &lv[L][4]);
                                }
                                tc::tmem_wait_ld();
                                if (hf == 1) release_acc(s);      // last read of this accumulator set
                                if (my == kHist) {
#pragma unroll
                                    for (int i0 = 0; i0 < 8; i0 += 4) {        // four independent mass evaluations at a time
                                        unsigned long long delta[4];
                                        bool in[4];
                                        bool any_in = false;
#pragma unroll
                                        for (int u = 0; u < 4; ++u) {
                                            const int i = i0 + u;
                                            const int hi = (int)lv[0][i] * 256 + (int)lv[1][i];
                                            const int lw = (int)lv[2][i] * 256 + (int)lv[3][i];
                                            delta[u] = (unsigned long long)(VA - ((long long)hi * 65536 + lw));
                                            in[u] = colh + (i0 >> 2) * 16 + u < n && delta[u] - lo <= span;
                                            any_in |= in[u];
                                        }
                                        if (!any_in) continue;
                                        unsigned long long m[4];
#pragma unroll
                                        for (int u = 0; u < 4; ++u) m[u] = kByCount ? 1ull : mass38(to_double(delta[u]) * neg_f);
#pragma unroll
                                        for (int u = 0; u < 4; ++u) {
                                            if (in[u]) {
                                                const unsigned long long bq = (delta[u] - lo) >> sh;
                                                const int b = bq > 63ull ? 63 : (int)bq;
                                                atomicAdd(&hist[b * 128], (m[u] << 13) | 1ull);
                                            }
                                        }
                                    }
                                } else if (my == kCollect) {
#pragma unroll
                                    for (int i = 0; i < 8; ++i) {
                                        const int hi = (int)lv[0][i] * 256 + (int)lv[1][i];
                                        const int lw = (int)lv[2][i] * 256 + (int)lv[3][i];
                                        const unsigned long long delta = (unsigned long long)(VA - ((long long)hi * 65536 + lw));
                                        const int j = colh + (i >> 2) * 16 + (i & 3);
                                        const bool in_row = j < n;
                                        if (in_row && delta - lo <= span) {
                                            const int slot = atomicAdd(&sm.cand_cnt[r], 1);
                                            if (slot < kCandCap) cand[slot * 128] = (delta << 12) | (unsigned long long)j;
                                        }
                                        bits |= ((in_row && delta < lo) ? 1u : 0u) << ((i >> 2) * 16 + part * 4 + (i & 3));
                                    }
                                }
                            } else if (hf == 1) {
                                release_acc(s);
                            }
                            if (!warp_idle && my == kCollect && bits) {
                                const int wd = ct * 2 + hf;
                                atomicOr(mask_row + (size_t)wd * kTileRows, bits);
                                if (bm_row) atomicOr(bm_row + wd, bits);
                                atomicAdd(&sm.row_count[r], __popc(bits));
                            }
                            if (!warp_idle) {
                                const uint32_t u = __reduce_or_sync(0xffffffffu, bits);
                                if (lane == 0 && u) atomicOr(&sm.tile_union[t_par][ct * 2 + hf], u);
                            }
                        }
                    }
                    if (!ok) break;
                    // ---------------- end of the pass: the row's four threads combine (three barriers, whatever the rows do)
                    if (!(ok = sync_rows())) break;               // A: histogram / candidate list complete
                    int n_cand = 0;
                    if (my == kHist) {
                        unsigned long long ps = 0ull;
#pragma unroll
                        for (int b = 0; b < 16; ++b) ps += hist[(part * 16 + b) * 128] >> 13;
                        sm.part[part][r] = ps;
                    } else if (my == kCollect) {
                        n_cand = sm.cand_cnt[r];
                        if (n_cand <= kCandCap)
                            for (int k = part; k < n_cand; k += 4)
                                hist[k * 128] = kByCount ? 1ull : mass38(to_double(cand[k * 128] >> 12) * neg_f);
                    }
                    if (!(ok = sync_rows())) break;               // B: partial sums / candidate masses visible
                    if (my == kHist) {
                        unsigned long long p4[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) p4[k] = sm.part[k][r];
                        if (first_level) {                        // Z and the target
                            const unsigned long long z = (p4[0] + p4[1]) + (p4[2] + p4[3]);
                            target = kByCount ? (z < (unsigned long long)g.top_k ? z : (unsigned long long)g.top_k)
                                              : (unsigned long long)ceil((double)z * g.top_p);
                            if (target == 0ull) target = 1ull;
                        }
                        unsigned long long cum = base;
                        int kk = 3;
#pragma unroll
                        for (int k = 0; k < 3; ++k)
                            if (kk == 3 && cum + p4[k] >= target) kk = k; else if (kk == 3) cum += p4[k];
                        if (part == kk) {                         // the crossing bucket is one of mine
                            int cb = 15, cnt = 0;
                            for (int b = 0; b < 16; ++b) {
                                const unsigned long long e = hist[(part * 16 + b) * 128];
                                if (cum + (e >> 13) >= target || b == 15) { cb = b; cnt = (int)(e & 8191ull); break; }
                                cum += e >> 13;
                            }
                            sm.res_base[r] = cum;
                            sm.res_cb[r] = (part * 16 + cb) | (cnt << 8);
                        }
#pragma unroll
                        for (int b = 0; b < 16; ++b) hist[(part * 16 + b) * 128] = 0ull;   // ready for the next histogram pass
                    } else if (my == kCollect) {
                        // the crossing cube among the collected ones: the smallest key whose mass, added to
                        // that of all smaller keys and of everything above the interval, reaches the target
                        unsigned long long best = ~0ull;
                        if (n_cand <= kCandCap) {
                            for (int i = part; i < n_cand; i += 4) {
                                const unsigned long long ki = cand[i * 128];
                                unsigned long long acc = base;
                                for (int k = 0; k < n_cand; ++k) acc += cand[k * 128] <= ki ? hist[k * 128] : 0ull;
                                if (acc >= target && ki < best) best = ki;
                            }
                        }
                        sm.part[part][r] = best;
                    }
                    if (!(ok = sync_rows())) break;               // C: results visible
                    if (my == kHist) {
                        ++hist_passes;
                        const int rc = sm.res_cb[r];
                        const int cb = rc & 63, cnt = rc >> 8;
                        base = sm.res_base[r];
                        const bool open_end = span == kOpen && cb == 63;   // the crossing lies beyond the window
                        lo += (unsigned long long)cb << sh;
                        if (!open_end) {
                            span = (1ull << sh) - 1ull;
                            if (span == 0ull || cnt <= kCandCap) state = kCollect;
                            else sh = sh >= 6 ? sh - 6 : 0;
                        } else if (cnt <= kCandCap) {
                            state = kCollect;
                        }
                        first_level = false;
                        if (state == kCollect && cnt > kCandCap) { state = kDone; give_up = true; }   // more exact ties than slots
                        if (state == kHist && hist_passes >= kMaxHistPasses) { state = kDone; give_up = true; }
                    } else if (my == kCollect) {
                        if (n_cand > kCandCap) {
                            give_up = true;
                        } else {
                            unsigned long long best = sm.part[0][r];
#pragma unroll
                            for (int k = 1; k < 4; ++k) best = min(best, sm.part[k][r]);
                            int added = 0;
                            for (int k = part; k < n_cand; k += 4) {
                                const unsigned long long kk = cand[k * 128];
                                if (kk <= best) {
                                    const int j = (int)(kk & 4095ull);
                                    const uint32_t bit = 1u << (j & 31);
                                    atomicOr(mask_row + (size_t)(j >> 5) * kTileRows, bit);
                                    if (bm_row) atomicOr(bm_row + (j >> 5), bit);
                                    atomicOr(&sm.tile_union[t_par][j >> 5], bit);
                                    ++added;
                                }
                            }
                            if (added) atomicAdd(&sm.row_count[r], added);
                            for (int k = part; k < kCandCap; k += 4) hist[k * 128] = 0ull;   // the masses kept there
                        }
                        state = kDone;
                    }
                    // ---------------- publish: does any row need a histogram pass after the next pass?
                    const int d = d0 + fpass;
                    if (state == kHist) *reinterpret_cast<volatile int32_t*>(&sm.need[d & 3]) = d + 1;
                    __threadfence_block();
                    __syncwarp();
                    if (lane == 0) tc::mbar_arrive(&sm.decided[d & 3]);
                    ++fpass;
                    bool more = true;
                    if (fpass >= 2) more = another_pass(d0 + fpass - 2, ok);
                    if (!ok || !more) break;
                }
                if (!ok) break;
                d0 += fpass;
                ++n_done;
            }
            // ---------------- end of the tile: union words, counts, rows handed over
            if (!(ok = sync_selection())) break;
            if (part == 0) {
                if (extra && sel_count) sel_count[raster_row] = sm.row_count[r];
                sm.row_count[r] = 0;
                sm.cand_cnt[r] = 0;
                if (give_up) {
                    const uint32_t slot = atomicAdd(fallback_count, 1u);
                    fallback_rows[slot] = (int32_t)(gt_cap * kTileRows + r);
                }
            } else if (part == 1 && r < g.n_words) {
                tile_union[gt_cap * g.n_words + r] = sm.tile_union[t_par][r];
                sm.tile_union[t_par][r] = 0u;             // this buffer is used again by the tile after the next
            }
        }
    }
    // ---------------------------------------------------------------- teardown
    tc::tc_fence_before_sync();
    __syncthreads();
    if (tid == 0 && sm.abort_flag) atomicExch(status, 6);
    if (warp == kProducerWarp) tc::tmem_dealloc<512>(tbase);
}

// p >= 1 without Top-K: every candidate cube is selected (Eq. 2 with p = 1).  grid (tiles of the call, Hq, B),
// 128 threads = rows of the tile.
__global__ void __launch_bounds__(128) select_all_kernel(Geom g, uint32_t* __restrict__ tile_mask,
                                                         uint32_t* __restrict__ tile_union, uint32_t* __restrict__ sel_bitmap,
                                                         int32_t* __restrict__ sel_count) {
    const int tile = blockIdx.x + g.tile_begin, h = blockIdx.y, b = blockIdx.z, r = threadIdx.x;
    const int pos = tile * kTileRows + r;
    const bool live = slot_live(g, pos);
    const int n = live ? n_candidates(g, pos) : 0;
    const size_t gt_cap = (size_t)(b * g.Hq + h) * g.n_tiles_cap + tile;
    const size_t raster_row = live ? (size_t)(b * g.Hq + h) * g.S_io + (pos_to_io(g, pos) - g.pos_begin) : 0;
    const int n_max = tile_max_candidates(g, tile);
    for (int w = 0; w < g.n_words; ++w) {
        const int rem = n - w * 32;
        const uint32_t word = rem >= 32 ? 0xffffffffu : (rem > 0 ? (1u << rem) - 1u : 0u);
        tile_mask[(gt_cap * g.n_words + w) * kTileRows + r] = word;
        if (sel_bitmap && live) sel_bitmap[raster_row * g.n_words + w] = word;
        if (r == 0) {
            const int remx = n_max - w * 32;
            tile_union[gt_cap * g.n_words + w] = remx >= 32 ? 0xffffffffu : (remx > 0 ? (1u << remx) - 1u : 0u);
        }
    }
    if (sel_count && live) sel_count[raster_row] = n;
}

}  // namespace adaspark
