// K4: gathered flash-style attention on the 5th-generation tensor cores (Eq. 3; un-permute of
// Algorithm 1 fused into the epilogue).
//
// One CTA = one "pair tile": 256 consecutive cube-major query rows of one query head, handled as
// two 128-row MMA tiles that ping-pong on the tensor core.  Roles (384 threads):
//   warps 0-3   softmax of tile 0 (thread = query row = TMEM lane)
//   warps 4-7   softmax of tile 1
//   warp  8     TMA producer: Q tiles once, then K / V^T tiles of the needed key blocks
//   warp  9     MMA issuer: S_t = Q_t K^T (operands in shared memory), O_t += P_t V (P in TMEM)
//   warps 10-11 idle; they complete the third warpgroup so that it can hand registers to the
//               softmax warpgroups (setmaxnreg), which hold a whole 128-column score row each
// Key blocks (64 cube-major positions) are visited in pairs (128 keys per step).  A block is
// needed if any row of the pair tile selected a cube inside it or if it overlaps the tile's local
// range (own cubes / text prefix).  Each softmax thread masks its own row: one selection bit per
// (row, cube) for blocks before the local range, the exact per-key rule inside it.
//
// TMEM (512 columns): tile t owns [256t, 256t+128) for S_t (fp32) -- P_t (bf16 pairs) overwrites
// its first 64 columns -- and [256t+128, 256t+128+D) for O_t.  The issue order
//   S0(0) S1(0) | PV0(j) S0(j+1) PV1(j) S1(j+1) ...
// lets the softmax of one tile overlap the MMAs of the other, and makes "S_t(j+1) ready" imply
// "PV_t(j) finished", so the lazy rescale of O_t needs no extra barrier.
#pragma once
#include "tc_common.cuh"

namespace adaspark {

constexpr int kTcThreads = 384;
constexpr int kSoftmaxRegs = 216;   // per-thread registers of the softmax warpgroups after setmaxnreg
constexpr int kHelperRegs = 72;     // ... of the producer / MMA warpgroup
// setmaxnreg only moves registers inside what the CTA got at launch: 384 threads x 168 registers (the
// compile-time bound of __launch_bounds__(384, 1)).  A request beyond that blocks forever.
static_assert(8 * 32 * kSoftmaxRegs + 4 * 32 * kHelperRegs <= kTcThreads * 168, "setmaxnreg must stay inside the CTA's launch allocation");
constexpr int kPairRows = 256;
// Largest score bound B (log2 units) up to which a row's softmax reference is fixed in advance.  Every score lies
// in [-B, B], so every weight 2^(s - B) is at least 2^-2B = 2^-96: nothing underflows, and 30 binades remain
// above the smallest normal fp32 for the products with V.
constexpr float kFixedRefMax = 48.f;
constexpr int kMaxBlockWords = 1024;   // up to 32768 key blocks (2M positions) per sequence

template <int D>
struct TcAttnSmem {
    __nv_bfloat16 q[2][D / 64][128][64];      // [tile][d panel][row][64 d]
    __nv_bfloat16 k[2][D / 64][128][64];      // [stage][d panel][key (2 blocks)][64 d]
    __nv_bfloat16 v[2][2][D][64];             // [stage][block][d][64 keys]  (V^T)
    uint32_t blk_words[kMaxBlockWords];       // bit kb set <=> key block kb is visited
    uint32_t union_words[128];                // OR of the 256 rows' selection words
    uint64_t q_full, k_full[2], k_empty[2], v_full[2], v_empty[2], s_full[2], p_half[2][2], o_final;
    uint32_t tmem_base;
    int abort_flag;
    int n_needed;                             // number of visited key blocks
};

// Iterates the set bits of blk_words in ascending order.
struct BlockIter {
    const uint32_t* words;
    int wi;
    uint32_t cur;
    __device__ __forceinline__ BlockIter(const uint32_t* w) : words(w), wi(0), cur(w[0]) {}
    __device__ __forceinline__ int next() {   // caller guarantees a set bit remains
        while (cur == 0) cur = words[++wi];
        int b = __ffs(cur) - 1;
        cur &= cur - 1;
        return wi * 32 + b;
    }
};

template <int D>
__global__ void __launch_bounds__(kTcThreads, 1) attn_prefill_tc_kernel(
    Geom g, const __grid_constant__ CUtensorMap tmQ, const __nv_bfloat16* __restrict__ q, const __grid_constant__ CUtensorMap tmK,
    const __grid_constant__ CUtensorMap tmV, const uint32_t* __restrict__ tile_mask,
    const uint32_t* __restrict__ tile_union, const uint32_t* __restrict__ slot_valid, const uint32_t* __restrict__ pair_mode,
    int n_pairs_cap, float2* __restrict__ ml_local, const uint32_t* __restrict__ key_norm2_bits, __nv_bfloat16* __restrict__ out,
    unsigned long long* __restrict__ executed_blocks, uint32_t* __restrict__ max_tile_blocks, int32_t* __restrict__ status) {
    extern __shared__ unsigned char tc_smem_raw[];
    TcAttnSmem<D>& sm = *reinterpret_cast<TcAttnSmem<D>*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kPanels = D / 64;
    constexpr int kQKSteps = D / 16;                            // k-steps of S = Q K^T
    constexpr uint32_t kIdescS = tc::make_idesc_bf16(128, 128);  // S tile: 128 rows x 128 keys
    constexpr uint32_t kIdescO = tc::make_idesc_bf16(128, D);    // O tile: 128 rows x D
    constexpr uint32_t kKBytes = 128 * D * 2, kVBytes = 2 * D * 64 * 2;

    const int n_pairs = (g.S + kPairRows - 1) / kPairRows;
    // 1-D grid, pair-major: the late (long) pair tiles of every head and batch entry start first
    const int n_hb = g.Hq * g.B;
    const int pair = n_pairs - 1 - (int)blockIdx.x / n_hb;
    const int hb = (int)blockIdx.x - (n_pairs - 1 - pair) * n_hb;
    const int b = hb / g.Hq, h = hb - b * g.Hq, gk = h / g.G;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int pair_pos0 = pair * kPairRows;
    const int pair_end = min(pair_pos0 + kPairRows, g.S);       // exclusive
    // key blocks that can matter: up to the pair's own end, and for a pair with video rows also the blocks
    // of the text prefix (attended by every video row)
    const int prefix_blk0 = g.S_v / kBlockTok, prefix_blk1 = (g.S_v + g.n_prefix + kBlockTok - 1) / kBlockTok;
    const bool sees_prefix = g.n_prefix > 0 && pair_pos0 < g.S_v;
    const int n_blk_own = (pair_end + kBlockTok - 1) / kBlockTok;
    const int n_blk = sees_prefix ? max(n_blk_own, prefix_blk1) : n_blk_own;
    const int first_local_blk = pair_first_local_blk(g, pair_pos0);
    // A pair whose selected cubes go through the query-gather kernels (attn_gather.cuh) visits only its local
    // range and the text prefix here and leaves (reference exponent, sum) of every row for the merge.
    const bool gathered = pair_mode != nullptr && __ldg(pair_mode + (size_t)(b * g.Hq + h) * n_pairs_cap + pair) != 0u;

    // ---------------------------------------------------------------- set-up
    if (tid == 0) {
        tc::mbar_init(&sm.q_full, 1);
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(&sm.k_full[i], 1);
            tc::mbar_init(&sm.k_empty[i], 1);
            tc::mbar_init(&sm.v_full[i], 1);
            tc::mbar_init(&sm.v_empty[i], 1);
            tc::mbar_init(&sm.s_full[i], 1);
            tc::mbar_init(&sm.p_half[i][0], 128);
            tc::mbar_init(&sm.p_half[i][1], 128);
        }
        tc::mbar_init(&sm.o_final, 1);
        sm.abort_flag = 0;
        tc::fence_barrier_init();
    }
    if (warp == 8) {
        tc::tmem_alloc<512>(&sm.tmem_base);
        if (lane == 0) {
            tc::prefetch_tensormap(&tmQ);
            tc::prefetch_tensormap(&tmK);
            tc::prefetch_tensormap(&tmV);
        }
    }
    __syncthreads();                                            // barriers initialised
    if (warp == 8) {
        // The Q tiles do not depend on the block plan: their load overlaps the union computation below.  They come
        // straight from the caller's tensor [B, S_io, Hq, D]: the video rows of a tile are whole boxes of a cube's
        // window (or the cubes themselves, below 128 tokens) in the (head x d, x, y, t, batch) view of that tensor,
        // which one 5-D TMA load per box and 64-element panel turns into cube-major rows (a coordinate beyond the
        // grid reads zeros: the empty slots of a boundary cube); text rows and the slots beyond the sequence,
        // a few tiles per head, are copied by the warp's lanes.
        const int rpb = min(g.C, 128);                            // rows per box
        uint32_t tx_bytes = 0;
#pragma unroll 1
        for (int t = 0; t < 2; ++t) {
            const int p0 = pair_pos0 + t * 128;
            const int n_vid = max(0, min(p0 + 128, g.S_v) - p0);  // video slots of the tile (a multiple of rpb or of C)
            for (int idx = lane; idx < (128 - n_vid) * (D / 8); idx += 32) {
                const int row = n_vid + idx / (D / 8), c = idx % (D / 8);
                const int pos = p0 + row;
                uint4 val = make_uint4(0u, 0u, 0u, 0u);
                if (pos < g.S) val = __ldg(reinterpret_cast<const uint4*>(q + (io_row(g, b, pos) * g.Hq + h) * D) + c);
                *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(&sm.q[t][c >> 3][0][0]) + sw128(row, c & 7)) = val;
            }
            tx_bytes += (uint32_t)n_vid * D * 2;
        }
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");   // the copied rows are read by the tensor core
        __syncwarp();
        if (lane == 0) {
            if (tx_bytes) tc::mbar_arrive_expect_tx(&sm.q_full, tx_bytes);
            else tc::mbar_arrive(&sm.q_full);
            for (int t = 0; t < 2; ++t) {
                const int p0 = pair_pos0 + t * 128;
                const int n_vid = max(0, min(p0 + 128, g.S_v) - p0);
                for (int r = 0; r < n_vid; r += rpb) {
                    const int pos = p0 + r;
                    const int c = pos >> g.c_shift, r0 = pos & (g.C - 1);
                    int cx, cy, cb, tt;
                    g.div_nW.divmod(c, tt, cx);
                    g.div_nH.divmod(tt, cb, cy);
                    const int x = cx * g.cw + (r0 & (g.cw - 1));
                    const int y = cy * g.ch + ((r0 >> g.cw_shift) & (g.ch - 1));
                    const int fr = cb * g.ct + (r0 >> (g.cw_shift + g.ch_shift)) - g.frame_begin;
                    for (int p = 0; p < kPanels; ++p)
                        tc::tma_load_5d(&sm.q[t][p][r][0], &tmQ, h * D + p * 64, x, y, fr, b, &sm.q_full);
                }
            }
        }
    }
    // union of the selection words of the 256 rows = OR of the two tiles' union words (written by the
    // selection kernel)
    for (int w = tid; w < g.n_words; w += kTcThreads) {
        uint32_t u = 0;
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int tile = pair * 2 + t;
            if (tile < g.n_tiles) u |= __ldg(tile_union + ((size_t)(b * g.Hq + h) * g.n_tiles_cap + tile) * g.n_words + w);
        }
        sm.union_words[w] = u;
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    // block bitmap: one thread per word of 32 key blocks
    const int n_blk_words = (n_blk + 31) / 32;
    for (int wi = tid; wi < n_blk_words; wi += kTcThreads) {
        uint32_t bits = 0;
        if (g.c_shift == 6 && wi * 32 + 31 < first_local_blk) {   // (first_local_blk <= prefix_blk0)
            bits = gathered ? 0u : sm.union_words[wi];   // 64-token cubes: key block = cube, the word is the union word
        } else {
            for (int i = 0; i < 32; ++i) {
                int kb = wi * 32 + i;
                if (kb >= n_blk) break;
                bool need = (kb >= first_local_blk && kb < n_blk_own) || (sees_prefix && kb >= prefix_blk0);
                if (!need && !gathered) {
                    int c_lo = (kb * kBlockTok) >> g.c_shift, c_hi = (kb * kBlockTok + kBlockTok - 1) >> g.c_shift;
                    uint32_t span = c_hi - c_lo + 1;   // <= 4 cubes, aligned: never crosses a word
                    uint32_t m = (span >= 32 ? 0xffffffffu : ((1u << span) - 1u)) << (c_lo & 31);
                    need = (sm.union_words[c_lo >> 5] & m) != 0;
                }
                if (need) bits |= 1u << i;
            }
        }
        sm.blk_words[wi] = bits;
    }
    __syncthreads();
    if (warp == 0) {
        int cnt = 0;
        for (int wi = lane; wi < n_blk_words; wi += 32) cnt += __popc(sm.blk_words[wi]);
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (lane == 0) sm.n_needed = cnt;
    }
    __syncthreads();
    const int n_needed = sm.n_needed;
    const int n_steps = (n_needed + 1) / 2;                      // >= 1: the local range is never empty
    const uint32_t tbase = sm.tmem_base;
    volatile int* abort_flag = &sm.abort_flag;

    if (warp >= 8) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;\n" ::"n"(kHelperRegs));
    if (warp == 8) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const int kv_row0 = (b * g.Hkv + gk) * g.S_cap;
            const int v_row0 = (b * g.Hkv + gk) * g.n_kv_blocks_cap * D;
            BlockIter it(sm.blk_words);
            for (int j = 0; j < n_steps; ++j) {
                const int st = j & 1, u = j >> 1;
                const int kb_a = it.next();
                const int kb_b = (2 * j + 1 < n_needed) ? it.next() : kb_a;   // odd count: repeat, masked later
                if (!tc::mbar_wait(&sm.k_empty[st], (u & 1) ^ 1, abort_flag)) break;
                tc::mbar_arrive_expect_tx(&sm.k_full[st], kKBytes);
                for (int p = 0; p < kPanels; ++p) {
                    tc::tma_load_2d(&sm.k[st][p][0][0], &tmK, p * 64, kv_row0 + kb_a * kBlockTok, &sm.k_full[st]);
                    tc::tma_load_2d(&sm.k[st][p][64][0], &tmK, p * 64, kv_row0 + kb_b * kBlockTok, &sm.k_full[st]);
                }
                if (!tc::mbar_wait(&sm.v_empty[st], (u & 1) ^ 1, abort_flag)) break;
                tc::mbar_arrive_expect_tx(&sm.v_full[st], kVBytes);
                tc::tma_load_2d(&sm.v[st][0][0][0], &tmV, 0, v_row0 + kb_a * D, &sm.v_full[st]);
                tc::tma_load_2d(&sm.v[st][1][0][0], &tmV, 0, v_row0 + kb_b * D, &sm.v_full[st]);
            }
        }
    } else if (warp == 9) {
        // ------------------------------------------------------------ MMA issuer
        // The whole warp runs the loop and one elected lane issues: with every operand warp-uniform the
        // thread gets a 128x128x16 MMA accepted every 85 - 90 cycles; from a branch entered by lane 0 alone
        // it was 113 - 125 (the tensor core needs 64).
        {
            // descriptor low halves of the tile bases; a k-step of 16 elements advances 32 bytes
            // inside a 64-element panel (128-byte rows), panels / key blocks are 128 rows apart
            constexpr uint32_t kPanelStep = (128 * 64 * 2) >> 4, kKStep = 32 >> 4;
            constexpr uint32_t kVBlockStep = (D * 64 * 2) >> 4;
            constexpr uint32_t kQTileStep = (uint32_t)sizeof(sm.q[0]) >> 4, kKStageStep = (uint32_t)sizeof(sm.k[0]) >> 4;
            constexpr uint32_t kVStageStep = (uint32_t)sizeof(sm.v[0]) >> 4;
            const uint32_t q_lo0 = __shfl_sync(0xffffffffu, tc::smem_desc_lo_sw128(smem_u32(&sm.q[0][0][0][0])), 0);
            const uint32_t k_lo0 = __shfl_sync(0xffffffffu, tc::smem_desc_lo_sw128(smem_u32(&sm.k[0][0][0][0])), 0);
            const uint32_t v_lo0 = __shfl_sync(0xffffffffu, tc::smem_desc_lo_sw128(smem_u32(&sm.v[0][0][0][0])), 0);
            const uint32_t tb = __shfl_sync(0xffffffffu, tbase, 0);
            const int steps = __shfl_sync(0xffffffffu, n_steps, 0);
            auto issue_s = [&](int t, int st) {   // S_t = Q_t K(st)^T
                const uint32_t qa = q_lo0 + t * kQTileStep, kb = k_lo0 + st * kKStageStep, dst = tb + t * 256;
                tc::umma_ss_c<false>(dst, tc::smem_desc_from_halves(qa, tc::kSmemDescHiSw128),
                                     tc::smem_desc_from_halves(kb, tc::kSmemDescHiSw128), kIdescS);
#pragma unroll
                for (int ks = 1; ks < kQKSteps; ++ks) {
                    const uint32_t off = (ks >> 2) * kPanelStep + (ks & 3) * kKStep;
                    tc::umma_ss_c<true>(dst, tc::smem_desc_from_halves(qa + off, tc::kSmemDescHiSw128),
                                        tc::smem_desc_from_halves(kb + off, tc::kSmemDescHiSw128), kIdescS);
                }
            };
            // O_t (+)= P_t V(st), keys [64 half, 64 half + 64): the two halves are issued separately so
            // that the first can start while the softmax warps still produce the second
            auto issue_pv = [&](int t, int st, int half, bool first) {
                const uint32_t vb = v_lo0 + st * kVStageStep + half * kVBlockStep, dst = tb + t * 256 + 128;
                const uint32_t src = tb + t * 256 + half * 32;
                tc::umma_ts(dst, src, tc::smem_desc_from_halves(vb, tc::kSmemDescHiSw128), kIdescO, !first);
#pragma unroll
                for (int ks = 1; ks < 4; ++ks)
                    tc::umma_ts_c<true>(dst, src + ks * 8, tc::smem_desc_from_halves(vb + ks * kKStep, tc::kSmemDescHiSw128), kIdescO);
            };
            bool ok = tc::mbar_wait_warp(&sm.q_full, 0, abort_flag) && tc::mbar_wait_warp(&sm.k_full[0], 0, abort_flag);
            if (ok) {
                tc::tc_fence_after_sync();
                if (tc::elect_one()) {
                    issue_s(0, 0);
                    tc::umma_commit(&sm.s_full[0]);
                    issue_s(1, 0);
                    tc::umma_commit(&sm.s_full[1]);
                    tc::umma_commit(&sm.k_empty[0]);
                }
                __syncwarp();
            }
            for (int j = 0; ok && j < steps; ++j) {
                const int st = j & 1, u = j >> 1;
                const bool more = j + 1 < steps;
                const int st1 = (j + 1) & 1, u1 = (j + 1) >> 1;
                if (!(ok = tc::mbar_wait_warp(&sm.v_full[st], u & 1, abort_flag))) break;
                if (!(ok = tc::mbar_wait_warp(&sm.p_half[0][0], j & 1, abort_flag))) break;
                tc::tc_fence_after_sync();
                if (tc::elect_one()) issue_pv(0, st, 0, j == 0);
                __syncwarp();
                if (!(ok = tc::mbar_wait_warp(&sm.p_half[0][1], j & 1, abort_flag))) break;
                tc::tc_fence_after_sync();
                if (more && !(ok = tc::mbar_wait_warp(&sm.k_full[st1], u1 & 1, abort_flag))) break;
                tc::tc_fence_after_sync();
                if (tc::elect_one()) {
                    issue_pv(0, st, 1, false);
                    if (more) {
                        issue_s(0, st1);
                        tc::umma_commit(&sm.s_full[0]);
                    }
                }
                __syncwarp();
                if (!(ok = tc::mbar_wait_warp(&sm.p_half[1][0], j & 1, abort_flag))) break;
                tc::tc_fence_after_sync();
                if (tc::elect_one()) issue_pv(1, st, 0, j == 0);
                __syncwarp();
                if (!(ok = tc::mbar_wait_warp(&sm.p_half[1][1], j & 1, abort_flag))) break;
                tc::tc_fence_after_sync();
                if (tc::elect_one()) {
                    issue_pv(1, st, 1, false);
                    tc::umma_commit(&sm.v_empty[st]);
                    if (more) {
                        issue_s(1, st1);
                        tc::umma_commit(&sm.s_full[1]);
                        tc::umma_commit(&sm.k_empty[st1]);
                    }
                }
                __syncwarp();
            }
            if (ok && tc::elect_one()) tc::umma_commit(&sm.o_final);
            __syncwarp();
        }
    } else if (warp < 8) {
        // ------------------------------------------------------------ softmax warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;\n" ::"n"(kSoftmaxRegs));
        const int t = warp >> 2;                                  // tile of this warpgroup
        const int row = (warp & 3) * 32 + lane;                   // row inside the tile = TMEM lane
        const int tile = pair * 2 + t;
        const int pr = pair_pos0 + t * 128 + row;                 // cube-major position of the row
        const uint32_t lane_addr = tbase + ((uint32_t)((warp & 3) * 32) << 16) + t * 256;
        const bool tile_live = tile < g.n_tiles;
        const uint32_t* my_mask = tile_mask + mask_index(g, b, h, tile_live ? tile : 0, 0, row);
        const float scale_log2 = g.scale_log2;
        int cached_w = -1;
        uint32_t cached_word = 0;
        auto get_word = [&](int w) -> uint32_t {
            if (w != cached_w) {
                cached_w = w;
                cached_word = tile_live ? my_mask[(size_t)w * kTileRows] : 0u;
            }
            return cached_word;
        };
        float m_ref = -INFINITY, l_sum = 0.f;
        // Reference fixed in advance.  |s| <= |q| |k| for every key, so with B = |q| max|k| scale (in log2 units;
        // the largest key norm of the head comes from the re-layout kernel) 2^(s scale - B) can never
        // overflow: the row needs no maximum and no rescaling of O.  What it costs is range at the small end
        // (a weight may be as low as 2^-2B), so the rows of the warp take this path only if all their bounds
        // are small; otherwise, and when not every attended key went through this call's re-layout, the
        // running maximum below decides as before.
        bool fixed_ref = false;
        if (key_norm2_bits != nullptr) {
            float bound = INFINITY;
            if (tc::mbar_wait(&sm.q_full, 0, abort_flag)) {
                float q2 = 0.f;
#pragma unroll
                for (int c = 0; c < D / 8; ++c) {
                    const uint4 qv = *reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(&sm.q[t][c >> 3][0][0]) + sw128(row, c & 7));
                    const uint32_t w[4] = {qv.x, qv.y, qv.z, qv.w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xffff0000u);
                        q2 = fmaf(lo, lo, fmaf(hi, hi, q2));
                    }
                }
                const float k2 = __uint_as_float(__ldg(key_norm2_bits + b * g.Hkv + gk));
                bound = sqrtf(q2 * k2) * scale_log2 * 1.01f + 0.01f;     // 1 % for the rounding of the norms and of s
            }
            fixed_ref = __all_sync(0xffffffffu, bound <= kFixedRefMax);
            if (fixed_ref) m_ref = bound;
        }
        BlockIter it(sm.blk_words);
        bool ok = true;
        for (int j = 0; j < n_steps; ++j) {
            const int kb_a = it.next();
            const bool has_b = 2 * j + 1 < n_needed;
            const int kb_b = has_b ? it.next() : kb_a;
            // ---- visibility of the 128 keys of this step for this row: one bit per key
            uint32_t amask[4];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int kb = hf ? kb_b : kb_a;
                const int pk0 = kb * kBlockTok;
                uint32_t m0 = 0, m1 = 0;
                if (hf == 1 && !has_b) {
                    // repeated block of an odd count: nothing visible
                } else if (kb < first_local_blk) {
                    const int cube0 = pk0 >> g.c_shift;
                    const uint32_t wbits = get_word(cube0 >> 5) >> (cube0 & 31);
                    if (g.c_shift >= 6) {
                        m0 = m1 = (wbits & 1u) ? 0xffffffffu : 0u;
                    } else if (g.c_shift == 5) {
                        m0 = (wbits & 1u) ? 0xffffffffu : 0u;
                        m1 = (wbits & 2u) ? 0xffffffffu : 0u;
                    } else {
                        m0 = ((wbits & 1u) ? 0x0000ffffu : 0u) | ((wbits & 2u) ? 0xffff0000u : 0u);
                        m1 = ((wbits & 4u) ? 0x0000ffffu : 0u) | ((wbits & 8u) ? 0xffff0000u : 0u);
                    }
                } else {
                    // local range: every aligned group of 16 keys lies in one cube or in the text
                    // (C >= 16 and S_v is a multiple of C), so the rule of Eq. 3 is closed-form per group
                    const uint32_t word = pk0 < g.S_v ? get_word((pk0 >> g.c_shift) >> 5) : 0u;
                    uint32_t gm[4];
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        const int pg = pk0 + q4 * 16;
                        // keys pg..pr; a video row sees the text prefix (slots S_v .. S_v + n_prefix) in full
                        const int n_causal = (pg >= g.S_v && pr < g.S_v) ? min(max(g.S_v + g.n_prefix - pg, 0), 16)
                                                                         : min(max(pr - pg + 1, 0), 16);
                        const uint32_t causal = (1u << n_causal) - 1u;
                        const int ck = pg >> g.c_shift;
                        const bool own = pg >= g.S_v || (pr < g.S_v && ck == (pr >> g.c_shift));
                        const uint32_t picked = (pg < g.S_v && ((word >> (ck & 31)) & 1u)) ? 0xffffu : 0u;
                        gm[q4] = own ? causal : picked;
                    }
                    m0 = gm[0] | (gm[1] << 16);
                    m1 = gm[2] | (gm[3] << 16);
                }
                if (g.ragged && pk0 < g.S_v && !(hf == 1 && !has_b)) {   // empty slots of boundary cubes are never attended
                    m0 &= __ldg(slot_valid + 2 * kb);
                    m1 &= __ldg(slot_valid + 2 * kb + 1);
                }
                amask[hf * 2] = m0;
                amask[hf * 2 + 1] = m1;
            }
            // every 32-key chunk of every row of the warp fully visible or fully hidden?
            const bool uniform = __all_sync(0xffffffffu, (amask[0] + 1u <= 1u) && (amask[1] + 1u <= 1u) &&
                                                             (amask[2] + 1u <= 1u) && (amask[3] + 1u <= 1u));
            if (!(ok = tc::mbar_wait(&sm.s_full[t], j & 1, abort_flag))) break;
            tc::tc_fence_after_sync();
            uint32_t s[4][32];
#pragma unroll
            for (int c = 0; c < 4; ++c) tc::tmem_ld_32x32(lane_addr + c * 32, s[c]);
            tc::tmem_wait_ld();
            if (!fixed_ref) {
            // ---- row maximum over the visible keys
            float mx = -INFINITY;
            if (uniform) {
                float a[4][2];
#pragma unroll
                for (int c = 0; c < 4; ++c) a[c][0] = a[c][1] = -INFINITY;
#pragma unroll
                for (int i = 0; i < 8; ++i)          // eight independent chains
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        a[c][0] = fmax3(a[c][0], __uint_as_float(s[c][4 * i]), __uint_as_float(s[c][4 * i + 1]));
                        a[c][1] = fmax3(a[c][1], __uint_as_float(s[c][4 * i + 2]), __uint_as_float(s[c][4 * i + 3]));
                    }
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    mx = fmax3(mx, amask[c] ? a[c][0] : -INFINITY, amask[c] ? a[c][1] : -INFINITY);
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t am = amask[c];
                    float a0 = -INFINITY, a1 = -INFINITY;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        a0 = fmaxf(a0, ((am >> (2 * i)) & 1u) ? __uint_as_float(s[c][2 * i]) : -INFINITY);
                        a1 = fmaxf(a1, ((am >> (2 * i + 1)) & 1u) ? __uint_as_float(s[c][2 * i + 1]) : -INFINITY);
                    }
                    mx = fmax3(mx, a0, a1);
                }
            }
            const float mx_x = mx * scale_log2;                   // scale > 0: max commutes with it
            // ---- lazy rescale: move the reference only when it grows by more than 2^8
            const bool need = mx_x > m_ref + 8.f;                  // also true on the first visible key
            if (__any_sync(0xffffffffu, need)) {
                const float factor = need ? exp2f(m_ref - mx_x) : 1.f;   // 0 when nothing was visible before
                if (j > 0) {
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        tc::tmem_ld_32x32(lane_addr + 128 + c * 32, o);
                        tc::tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                        tc::tmem_st_32x32(lane_addr + 128 + c * 32, o);
                    }
                }
                l_sum *= factor;
                if (need) m_ref = mx_x;
            }
            }
            // ---- P = 2^(s*scale - m_ref) on visible keys, 0 elsewhere; bf16 pairs into TMEM
            const float neg_ref = -m_ref;                          // finite whenever a key is visible
            if (uniform) {
                // The scale-subtract and the row sums use the packed fp32x2 instructions: 10 instead of 14
                // instructions per four keys.
                unsigned long long psA = 0ull, psB = 0ull;             // two packed pairs of partial row sums
                const unsigned long long scale2 = pack_f32x2(scale_log2, scale_log2);
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float addend = amask[c] ? neg_ref : -INFINITY;   // 2^(-inf) = 0 hides the chunk
                    const unsigned long long add2 = pack_f32x2(addend, addend);
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const unsigned long long x01 = fma_f32x2(pack_f32x2(__uint_as_float(s[c][4 * i]), __uint_as_float(s[c][4 * i + 1])), scale2, add2);
                        const unsigned long long x23 = fma_f32x2(pack_f32x2(__uint_as_float(s[c][4 * i + 2]), __uint_as_float(s[c][4 * i + 3])), scale2, add2);
                        float x0, x1, x2, x3;
                        unpack_f32x2(x01, x0, x1);
                        unpack_f32x2(x23, x2, x3);
                        // one exponential in eight on the FMA pipe: a softmax warp running alone on its
                        // scheduler is bound by MUFU (8 cycles per warp-wide ex2) and by issue about equally
                        // (measured: 1/8 gains 2.5 %, 1/4 loses 1 %, 1/2 loses 6 %)
                        const float p0 = fast_exp2(x0), p1 = fast_exp2(x1), p2 = fast_exp2(x2), p3 = (i & 1) ? fma_exp2(x3) : fast_exp2(x3);
                        psA = add_f32x2(psA, pack_f32x2(p0, p1));
                        psB = add_f32x2(psB, pack_f32x2(p2, p3));
                        pk[2 * i] = pack_bf16x2(p0, p1);
                        pk[2 * i + 1] = pack_bf16x2(p2, p3);
                    }
                    tc::tmem_st_32x16(lane_addr + c * 16, pk);
                    if (c == 1) {                                   // first 64 keys of P are in place
                        tc::tmem_wait_st();
                        tc::tc_fence_before_sync();
                        tc::mbar_arrive(&sm.p_half[t][0]);
                    }
                }
                float a0, a1, b0, b1;
                unpack_f32x2(psA, a0, a1);
                unpack_f32x2(psB, b0, b1);
                l_sum += (a0 + a1) + (b0 + b1);
            } else {
                float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t am = amask[c];
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        float p0 = fast_exp2(fmaf(__uint_as_float(s[c][2 * i]), scale_log2, ((am >> (2 * i)) & 1u) ? neg_ref : -INFINITY));
                        float p1 = fast_exp2(fmaf(__uint_as_float(s[c][2 * i + 1]), scale_log2, ((am >> (2 * i + 1)) & 1u) ? neg_ref : -INFINITY));
                        ps0 += p0; ps1 += p1;
                        pk[i] = pack_bf16x2(p0, p1);
                    }
                    tc::tmem_st_32x16(lane_addr + c * 16, pk);
                    if (c == 1) {
                        tc::tmem_wait_st();
                        tc::tc_fence_before_sync();
                        tc::mbar_arrive(&sm.p_half[t][0]);
                    }
                }
                l_sum += ps0 + ps1;
            }
            tc::tmem_wait_st();
            tc::tc_fence_before_sync();
            tc::mbar_arrive(&sm.p_half[t][1]);
        }
        // ---- epilogue: O / l -> bf16 at the raster position of the row
        if (ok) ok = tc::mbar_wait(&sm.o_final, 0, abort_flag);
        if (ok) {
            tc::tc_fence_after_sync();
            const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
            const bool live = slot_live(g, pr);
            if (gathered && live) ml_local[(size_t)(b * g.Hq + h) * g.S_cap + pr] = make_float2(m_ref, l_sum);
            __nv_bfloat16* dst = out + ((live ? io_row(g, b, pr) : 0) * g.Hq + h) * D;
            uint32_t o[D / 32][32];                                // the whole output row in one round of loads
#pragma unroll
            for (int c = 0; c < D / 32; ++c) tc::tmem_ld_32x32(lane_addr + 128 + c * 32, o[c]);
            tc::tmem_wait_ld();
            // The row goes to shared memory (the Q / K tiles are no longer read: every MMA has completed)
            // and from there to its raster position as ONE 2*D-byte bulk copy: scattered 16-byte stores of
            // 32 different rows per instruction touch twice as many sectors (measured 1.7 % slower).
            constexpr int kRowPitch = 2 * D + 16;                 // bytes; keeps 16-byte alignment, spreads the banks
            unsigned char* srow = reinterpret_cast<unsigned char*>(&sm.q[0][0][0][0]) + (size_t)(t * 128 + row) * kRowPitch;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 val;
                    val.x = pack_bf16x2(__uint_as_float(o[c][8 * i + 0]) * inv, __uint_as_float(o[c][8 * i + 1]) * inv);
                    val.y = pack_bf16x2(__uint_as_float(o[c][8 * i + 2]) * inv, __uint_as_float(o[c][8 * i + 3]) * inv);
                    val.z = pack_bf16x2(__uint_as_float(o[c][8 * i + 4]) * inv, __uint_as_float(o[c][8 * i + 5]) * inv);
                    val.w = pack_bf16x2(__uint_as_float(o[c][8 * i + 6]) * inv, __uint_as_float(o[c][8 * i + 7]) * inv);
                    *reinterpret_cast<uint4*>(srow + (c * 4 + i) * 16) = val;
                }
            }
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
            if (live)
                asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;\n" ::"l"(dst), "r"(smem_u32(srow)), "n"(2 * D) : "memory");
            asm volatile("cp.async.bulk.commit_group;\n" ::: "memory");
            asm volatile("cp.async.bulk.wait_group.read 0;\n" ::: "memory");   // the row has left shared memory
        }
    }
    // ---------------------------------------------------------------- teardown
    tc::tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
        if (sm.abort_flag) atomicExch(status, 6);   // a bounded wait expired
        else {
            atomicAdd(executed_blocks, (unsigned long long)(2 * n_needed));
            atomicMax(max_tile_blocks, (uint32_t)n_needed);
        }
    }
    if (warp == 8) tc::tmem_dealloc<512>(tbase);
}

}  // namespace adaspark
