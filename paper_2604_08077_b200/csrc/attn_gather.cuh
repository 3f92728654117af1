// K4b: query-gather attention for sparse selections (Eq. 3 computed over the selected cubes only).
//
// The tile kernel (attn_prefill_tc.cuh) visits the union of the key blocks that the 256 rows of a pair of
// query tiles selected.  When the rows choose different cubes (independent queries) that union is nearly
// every block although each row keeps a few cubes: the executed work is the dense work.  This path turns
// the problem around.  For every 64-key block of the video it gathers, from all query tiles and all heads of
// the GQA group, the rows that selected a cube in it, and computes their attention over that block alone on
// the tensor cores: 128 gathered rows x 64 keys per item, S = Q K^T and O = P V as in the tile kernel.  Each
// (row, block) entry yields a partial result (reference exponent, sum, normalised output); a row's partials
// and the result of its local range (own cube, text, text prefix: still the tile kernel, which then skips
// the union) are merged by the softmax identity
//     out = sum_i w_i O_i / sum_i w_i,   w_i = l_i 2^(m_i - M),  M = max_i m_i.
// Executed work = selected work, at the price of 2 D + 8 bytes written and read per entry.
//
// Which pairs of query tiles take this path is decided on the device, per pair, from the counts the selection
// left: entries of the pair's rows (P) against key blocks in the pair's union (U), gathered iff
// P <= pairs_per_block * U.  If the entries of all such pairs exceed the capacity of the workspace, every
// pair stays on the tile kernel.  Kernels, in launch order:
//   gather_count_kernel   per pair: row counts, P, U, the decision, entries per key block (atomics)
//   gather_scan_kernel    one CTA: prefix sums over pairs and key blocks, work items of 128 entries
//   (attn_prefill_tc_kernel, which reads the decisions)
//   gather_fill_kernel    per pair: row -> first partial, entries into the lists of their key blocks
//   attn_gather_kernel    per item: gathered Q rows x one key block -> partials
//   gather_merge_kernel   per row: merge into `out`
// The order of a block's entries depends on the order of atomics, but an entry's arithmetic does not depend
// on its neighbours in the item, and a row merges its partials in ascending block order: results are
// deterministic.
#pragma once
#include "attn_prefill_tc.cuh"

namespace adaspark {

constexpr int kGatherThreads = 160;     // 4 softmax / gather warps + 1 TMA / MMA warp
constexpr int kGatherItemRows = 128;
constexpr uint32_t kEntryPosMask = 0x1fffffu;   // 21 bits of cube-major position (caches hold at most 2^21 rows)

// Pointers into the forward workspace and sizes (all filled by the host).
struct GatherWs {
    uint32_t* ctrl;        // [0] entries, [1] items, [2] pairs on this path (0 entries: the path is off)
    uint32_t* pair_mode;   // [B*Hq*n_pairs_cap] 1: the pair's selected cubes go through this path
    uint32_t* pair_cnt;    // entries of the pair's rows (0 when the pair stays on the tile kernel)
    uint32_t* pair_off;    // exclusive prefix sum of pair_cnt
    uint32_t* row_cnt;     // [B*Hq*S_cap] entries of a row
    uint32_t* row_ptr;     // index of the row's first partial
    uint32_t* col_cnt;     // [B*Hkv*n_cols] entries of a key block; zero at the start of a forward
    uint32_t* col_off;     // exclusive prefix sum of col_cnt
    uint32_t* col_cur;     // fill cursors; zero at the start of a forward
    uint2* items;          // (key block column, chunk of 128 entries)
    uint2* entries;        // x: pos | head in group << 21 | cube bits << 25;  y: index of the partial
    __nv_bfloat16* part_o; // [cap_entries][D] normalised partial outputs
    float2* part_ml;       // [cap_entries] (reference exponent in log2 units, sum)
    float2* ml_local;      // [B*Hq*S_cap] the same for the local range, written by the tile kernel
    uint32_t cap_entries;
    int n_cols;            // key blocks that hold video slots: ceil(S_v / 64)
    int n_pairs_cap;       // pairs of query tiles per (b, head): ceil(S_cap / 256)
    float pairs_per_block; // decision threshold (entries per union block)
};

// bit of the first cube of every 64-key block in which `word` has a selected cube (cubes of 16 / 32 tokens;
// for larger cubes a bit stands for 1 << (c_shift - 6) blocks and the word is returned as it is)
__device__ __forceinline__ uint32_t fold_to_blocks(uint32_t word, int c_shift) {
    if (c_shift == 5) return (word | (word >> 1)) & 0x55555555u;
    if (c_shift == 4) return (word | (word >> 1) | (word >> 2) | (word >> 3)) & 0x11111111u;
    return word;
}

struct PairItem {
    int pair, b, h, gk, pair_pos0, cube_lim, n_w;
    uint32_t last_keep;
};
// Pair of query tiles of CTA `bid` (pairs of the call's row window, all heads and batch entries) and the range
// of cubes that lie wholly before its local range: [0, cube_lim).
__device__ __forceinline__ PairItem pair_item(const Geom& g, int bid) {
    PairItem it;
    const int n_hb = g.Hq * g.B;
    it.pair = g.pos_begin / kPairRows + bid / n_hb;
    const int hb = bid - (bid / n_hb) * n_hb;
    it.b = hb / g.Hq;
    it.h = hb - it.b * g.Hq;
    it.gk = it.h / g.G;
    it.pair_pos0 = it.pair * kPairRows;
    it.cube_lim = (pair_first_local_blk(g, it.pair_pos0) * kBlockTok) >> g.c_shift;
    it.n_w = (it.cube_lim + 31) >> 5;
    it.last_keep = (it.cube_lim & 31) ? (1u << (it.cube_lim & 31)) - 1u : 0xffffffffu;
    return it;
}

// ------------------------------------------------------------------------------------------------ count
__global__ void __launch_bounds__(256) gather_count_kernel(Geom g, GatherWs ws, const uint32_t* __restrict__ tile_mask,
                                                           const uint32_t* __restrict__ tile_union) {
    __shared__ uint32_t red[2][8];
    __shared__ uint32_t s_mode;
    const PairItem it = pair_item(g, blockIdx.x);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bshift = max(g.c_shift - 6, 0);                   // log2(blocks per cube) for cubes of >= 64 tokens
    const int tile = it.pair * 2 + (warp >> 2), r = (warp & 3) * 32 + lane, pos = it.pair_pos0 + tid;
    const bool tile_ok = tile < g.n_tiles;
    const uint32_t* my = tile_mask + mask_index(g, it.b, it.h, tile_ok ? tile : 0, 0, r);
    const size_t bh = (size_t)(it.b * g.Hq + it.h);
    uint32_t cnt = 0;
    if (tile_ok)
        for (int w = 0; w < it.n_w; ++w) {
            uint32_t word = __ldg(my + (size_t)w * kTileRows);
            if (w == it.n_w - 1) word &= it.last_keep;
            cnt += (uint32_t)__popc(fold_to_blocks(word, g.c_shift)) << bshift;
        }
    if (pos < g.S_cap) ws.row_cnt[bh * g.S_cap + pos] = cnt;
    uint32_t ub = 0;
    for (int w = tid; w < it.n_w; w += 256) {
        uint32_t u = 0;
        for (int t = 0; t < 2; ++t)
            if (it.pair * 2 + t < g.n_tiles) u |= __ldg(tile_union + (bh * g.n_tiles_cap + it.pair * 2 + t) * g.n_words + w);
        if (w == it.n_w - 1) u &= it.last_keep;
        ub += (uint32_t)__popc(fold_to_blocks(u, g.c_shift)) << bshift;
    }
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    ub = __reduce_add_sync(0xffffffffu, ub);
    if (lane == 0) { red[0][warp] = cnt; red[1][warp] = ub; }
    __syncthreads();
    if (tid == 0) {
        uint32_t P = 0, U = 0;
        for (int i = 0; i < 8; ++i) { P += red[0][i]; U += red[1][i]; }
        const uint32_t mode = (P > 0 && (float)P <= ws.pairs_per_block * (float)U) ? 1u : 0u;
        const size_t slot = bh * ws.n_pairs_cap + it.pair;
        ws.pair_mode[slot] = mode;
        ws.pair_cnt[slot] = mode ? P : 0u;
        s_mode = mode;
    }
    __syncthreads();
    if (!s_mode || !tile_ok) return;
    // entries per key block: one atomic per (32 rows, block)
    uint32_t* col_cnt = ws.col_cnt + (size_t)(it.b * g.Hkv + it.gk) * ws.n_cols;
    for (int w = 0; w < it.n_w; ++w) {
        uint32_t word = __ldg(my + (size_t)w * kTileRows);
        if (w == it.n_w - 1) word &= it.last_keep;
        const uint32_t fw = fold_to_blocks(word, g.c_shift);
        uint32_t orw = __reduce_or_sync(0xffffffffu, fw);
        while (orw) {
            const int beta = __ffs(orw) - 1;
            orw &= orw - 1;
            const int n = __popc(__ballot_sync(0xffffffffu, (fw >> beta) & 1u));
            if (lane == 0) {
                const int cube = w * 32 + beta;
                if (g.c_shift >= 6) {
                    for (int i = 0; i < (1 << bshift); ++i) atomicAdd(col_cnt + ((size_t)cube << bshift) + i, (uint32_t)n);
                } else {
                    atomicAdd(col_cnt + (cube >> (6 - g.c_shift)), (uint32_t)n);
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------ scan
// exclusive prefix sum of one value per thread over a CTA of 1024 threads; *total receives the sum
__device__ __forceinline__ uint32_t cta_exclusive_scan_1024(uint32_t v, uint32_t* warp_sums, uint32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t inc = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += o;
    }
    __syncthreads();                       // warp_sums of the previous call are no longer read
    if (lane == 31) warp_sums[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        uint32_t s = warp_sums[lane], si = s;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t o = __shfl_up_sync(0xffffffffu, si, d);
            if (lane >= d) si += o;
        }
        warp_sums[lane] = si - s;          // exclusive over warps
        if (lane == 31) *total = si;
    }
    __syncthreads();
    return warp_sums[warp] + inc - v;
}

__global__ void __launch_bounds__(1024) gather_scan_kernel(Geom g, GatherWs ws) {
    __shared__ uint32_t warp_sums[32];
    __shared__ uint32_t total_s;
    __shared__ uint32_t big_col[1024], big_base[1024], big_n[1024];
    __shared__ uint32_t big_count;
    const int tid = threadIdx.x;
    const int pair0 = g.pos_begin / kPairRows, n_pairs = (g.S + kPairRows - 1) / kPairRows - pair0;
    const int n_hb = g.Hq * g.B;
    const int n_slots = n_pairs * n_hb;
    // ---- pairs: offsets of their rows' partials
    unsigned long long carry = 0ull;
    uint32_t n_on = 0;
    for (int base = 0; base < n_slots; base += 1024) {
        const int idx = base + tid;
        size_t slot = 0;
        uint32_t v = 0;
        if (idx < n_slots) {
            const int hb = idx / n_pairs, pr = idx - hb * n_pairs;
            slot = (size_t)hb * ws.n_pairs_cap + pair0 + pr;
            v = ws.pair_cnt[slot];
        }
        const uint32_t ex = cta_exclusive_scan_1024(v, warp_sums, &total_s);
        if (idx < n_slots) ws.pair_off[slot] = (uint32_t)(carry + ex);   // meaningless when the capacity check below fails
        n_on += (v != 0u);
        carry += total_s;
    }
    if (carry == 0ull || carry > (unsigned long long)ws.cap_entries) {
        // nothing to do, or more entries than the workspace holds: every pair stays on the tile kernel
        for (int idx = tid; idx < n_slots; idx += 1024) {
            const int hb = idx / n_pairs, pr = idx - hb * n_pairs;
            ws.pair_mode[(size_t)hb * ws.n_pairs_cap + pair0 + pr] = 0u;
        }
        if (tid == 0) { ws.ctrl[0] = 0u; ws.ctrl[1] = 0u; ws.ctrl[2] = 0u; }
        return;
    }
    n_on = __reduce_add_sync(0xffffffffu, n_on);
    __syncthreads();
    if ((tid & 31) == 0) warp_sums[tid >> 5] = n_on;
    __syncthreads();
    if (tid == 0) {
        uint32_t s = 0;
        for (int i = 0; i < 32; ++i) s += warp_sums[i];
        ws.ctrl[0] = (uint32_t)carry;
        ws.ctrl[2] = s;
    }
    // ---- key blocks: offsets of their entry lists and the work items (chunks of 128 entries)
    const int n_cols_all = g.B * g.Hkv * ws.n_cols;
    uint32_t ent_carry = 0, item_carry = 0;
    for (int base = 0; base < n_cols_all; base += 1024) {
        const int col = base + tid;
        const uint32_t v = col < n_cols_all ? ws.col_cnt[col] : 0u;
        const uint32_t chunks = (v + kGatherItemRows - 1) / kGatherItemRows;
        const uint32_t ex = cta_exclusive_scan_1024(v, warp_sums, &total_s);
        const uint32_t tot_e = total_s;
        const uint32_t exi = cta_exclusive_scan_1024(chunks, warp_sums, &total_s);
        const uint32_t tot_i = total_s;
        if (tid == 0) big_count = 0u;
        __syncthreads();
        if (col < n_cols_all) {
            ws.col_off[col] = ent_carry + ex;
            const uint32_t ib = item_carry + exi;
            if (chunks <= 32u) {
                for (uint32_t c = 0; c < chunks; ++c) ws.items[ib + c] = make_uint2((uint32_t)col, c);
            } else {
                const uint32_t k = atomicAdd(&big_count, 1u);
                big_col[k] = (uint32_t)col; big_base[k] = ib; big_n[k] = chunks;
            }
        }
        __syncthreads();
        const uint32_t nb = big_count;
        for (uint32_t k = 0; k < nb; ++k)
            for (uint32_t c = tid; c < big_n[k]; c += 1024) ws.items[big_base[k] + c] = make_uint2(big_col[k], c);
        ent_carry += tot_e;
        item_carry += tot_i;
        __syncthreads();
    }
    if (tid == 0) ws.ctrl[1] = item_carry;
}

// ------------------------------------------------------------------------------------------------ fill
__global__ void __launch_bounds__(256) gather_fill_kernel(Geom g, GatherWs ws, const uint32_t* __restrict__ tile_mask) {
    __shared__ uint32_t warp_tot[8];
    const PairItem it = pair_item(g, blockIdx.x);
    const size_t bh = (size_t)(it.b * g.Hq + it.h);
    const size_t slot = bh * ws.n_pairs_cap + it.pair;
    if (ws.ctrl[0] == 0u || ws.pair_mode[slot] == 0u) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bshift = max(g.c_shift - 6, 0);
    const int tile = it.pair * 2 + (warp >> 2), r = (warp & 3) * 32 + lane, pos = it.pair_pos0 + tid;
    const bool tile_ok = tile < g.n_tiles;
    // first partial of every row: prefix sum of the row counts inside the pair
    const uint32_t cnt = pos < g.S_cap ? ws.row_cnt[bh * g.S_cap + pos] : 0u;
    uint32_t inc = cnt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t o = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += o;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    uint32_t before = ws.pair_off[slot];
    for (int i = 0; i < warp; ++i) before += warp_tot[i];
    uint32_t ptr = before + inc - cnt;
    if (pos < g.S_cap) ws.row_ptr[bh * g.S_cap + pos] = ptr;
    if (!tile_ok) return;
    const uint32_t* my = tile_mask + mask_index(g, it.b, it.h, tile, 0, r);
    const size_t colbase = (size_t)(it.b * g.Hkv + it.gk) * ws.n_cols;
    const uint32_t ent_x = (uint32_t)pos | ((uint32_t)(it.h - it.gk * g.G) << 21);
    const uint32_t lt_mask = (1u << lane) - 1u;
    const int group = g.c_shift >= 6 ? 1 : (kBlockTok >> g.c_shift);    // cubes per key block (small cubes)
    for (int w = 0; w < it.n_w; ++w) {
        uint32_t word = __ldg(my + (size_t)w * kTileRows);
        if (w == it.n_w - 1) word &= it.last_keep;
        const uint32_t fw = fold_to_blocks(word, g.c_shift);
        uint32_t orw = __reduce_or_sync(0xffffffffu, fw);
        while (orw) {
            const int beta = __ffs(orw) - 1;
            orw &= orw - 1;
            const bool has = (fw >> beta) & 1u;
            const uint32_t m = __ballot_sync(0xffffffffu, has);
            const uint32_t n = (uint32_t)__popc(m), rank = (uint32_t)__popc(m & lt_mask);
            const int cube = w * 32 + beta;
            const int nblk = 1 << bshift;
            const size_t col0 = colbase + (g.c_shift >= 6 ? ((size_t)cube << bshift) : (size_t)(cube >> (6 - g.c_shift)));
            const uint32_t sub = g.c_shift >= 6 ? 0xfu : ((word >> beta) & ((1u << group) - 1u));
            for (int i = 0; i < nblk; ++i) {
                uint32_t start = 0;
                if (lane == 0) start = ws.col_off[col0 + i] + atomicAdd(ws.col_cur + col0 + i, n);
                start = __shfl_sync(0xffffffffu, start, 0);
                if (has) ws.entries[start + rank] = make_uint2(ent_x | (sub << 25), ptr + (uint32_t)i);
            }
            if (has) ptr += (uint32_t)nblk;
        }
    }
}

// ------------------------------------------------------------------------------------------------ attention
template <int D>
struct GatherSmem {
    __nv_bfloat16 q[D / 64][128][64];        // [d panel][gathered row][64 d], 128-byte swizzle
    __nv_bfloat16 k[2][D / 64][64][64];      // [stage][d panel][key][64 d]
    __nv_bfloat16 v[2][D][64];               // [stage][d][64 keys]  (V^T)
    uint2 ent[2][kGatherItemRows];
    uint64_t q_full, kv_full[2], s_full, p_full, o_full, ent_full;
    uint32_t tmem_base;
    int abort_flag;
};

template <int D>
__global__ void __launch_bounds__(kGatherThreads, 2) attn_gather_kernel(
    Geom g, GatherWs ws, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
    const __nv_bfloat16* __restrict__ q_cube, const uint32_t* __restrict__ slot_valid,
    unsigned long long* __restrict__ executed_blocks, int32_t* __restrict__ status) {
    extern __shared__ unsigned char gather_smem_raw[];
    GatherSmem<D>& sm = *reinterpret_cast<GatherSmem<D>*>((reinterpret_cast<uintptr_t>(gather_smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kPanels = D / 64, kQKSteps = D / 16, kChunks = D / 8;
    constexpr uint32_t kIdescS = tc::make_idesc_bf16(128, 64);   // S: 128 gathered rows x 64 keys
    constexpr uint32_t kIdescO = tc::make_idesc_bf16(128, D);    // O: 128 rows x D
    constexpr uint32_t kKVBytes = 64 * D * 2 * 2;
    constexpr int kTmemCols = 256;                               // S / P at [0, 64), O at [64, 64 + D)

    const uint32_t n_items = ws.ctrl[1];
    if (ws.ctrl[0] == 0u || blockIdx.x >= n_items) return;       // the path is off, or fewer items than CTAs
    const int my_items = (int)((n_items - blockIdx.x + gridDim.x - 1) / gridDim.x);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid == 0) {
        tc::mbar_init(&sm.q_full, kGatherItemRows);
        tc::mbar_init(&sm.kv_full[0], 1);
        tc::mbar_init(&sm.kv_full[1], 1);
        tc::mbar_init(&sm.s_full, 1);
        tc::mbar_init(&sm.p_full, kGatherItemRows);
        tc::mbar_init(&sm.o_full, 1);
        tc::mbar_init(&sm.ent_full, kGatherItemRows);
        sm.abort_flag = 0;
        tc::fence_barrier_init();
    }
    if (warp == 4) {
        tc::tmem_alloc<kTmemCols>(&sm.tmem_base);
        if (lane == 0) {
            tc::prefetch_tensormap(&tmK);
            tc::prefetch_tensormap(&tmV);
        }
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    const uint32_t tbase = sm.tmem_base;
    volatile int* abort_flag = &sm.abort_flag;

    // column of an item -> (batch x kv head, key block)
    auto item_col = [&](int i, int& bg, int& blk, uint32_t& first, int& n) {
        const uint2 iv = ws.items[blockIdx.x + (size_t)i * gridDim.x];
        bg = (int)(iv.x / (uint32_t)ws.n_cols);
        blk = (int)(iv.x - (uint32_t)bg * (uint32_t)ws.n_cols);
        first = ws.col_off[iv.x] + iv.y * kGatherItemRows;
        n = min(kGatherItemRows, (int)(ws.col_cnt[iv.x] - iv.y * kGatherItemRows));
    };

    if (warp == 4) {
        // ------------------------------------------------------------ TMA producer + MMA issuer (one thread)
        if (lane == 0) {
            auto load_kv = [&](int i) {
                int bg, blk, n;
                uint32_t first;
                item_col(i, bg, blk, first, n);
                const int st = i & 1;
                tc::mbar_arrive_expect_tx(&sm.kv_full[st], kKVBytes);
                for (int p = 0; p < kPanels; ++p)
                    tc::tma_load_2d(&sm.k[st][p][0][0], &tmK, p * 64, bg * g.S_cap + blk * kBlockTok, &sm.kv_full[st]);
                tc::tma_load_2d(&sm.v[st][0][0], &tmV, 0, (bg * g.n_kv_blocks_cap + blk) * D, &sm.kv_full[st]);
            };
            constexpr uint32_t kQPanelStep = (128 * 64 * 2) >> 4, kKPanelStep = (64 * 64 * 2) >> 4, kKStep = 32 >> 4;
            const uint32_t q_lo = tc::smem_desc_lo_sw128(smem_u32(&sm.q[0][0][0]));
            load_kv(0);
            for (int i = 0; i < my_items; ++i) {
                const int st = i & 1;
                const uint32_t k_lo = tc::smem_desc_lo_sw128(smem_u32(&sm.k[st][0][0][0]));
                const uint32_t v_lo = tc::smem_desc_lo_sw128(smem_u32(&sm.v[st][0][0]));
                if (!tc::mbar_wait(&sm.q_full, i & 1, abort_flag)) break;
                if (!tc::mbar_wait(&sm.kv_full[st], (i >> 1) & 1, abort_flag)) break;
                tc::tc_fence_after_sync();
#pragma unroll
                for (int ks = 0; ks < kQKSteps; ++ks) {
                    const uint32_t qo = (ks >> 2) * kQPanelStep + (ks & 3) * kKStep, ko = (ks >> 2) * kKPanelStep + (ks & 3) * kKStep;
                    tc::umma_ss(tbase, tc::smem_desc_from_halves(q_lo + qo, tc::kSmemDescHiSw128),
                                tc::smem_desc_from_halves(k_lo + ko, tc::kSmemDescHiSw128), kIdescS, ks > 0);
                }
                tc::umma_commit(&sm.s_full);
                if (!tc::mbar_wait(&sm.p_full, i & 1, abort_flag)) break;
                tc::tc_fence_after_sync();
                // every worker has passed the epilogue of item i-1, so that item's MMAs have completed and its
                // K / V stage can take the next block
                if (i + 1 < my_items) load_kv(i + 1);
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    tc::umma_ts(tbase + 64, tbase + ks * 8, tc::smem_desc_from_halves(v_lo + ks * kKStep, tc::kSmemDescHiSw128), kIdescO, ks > 0);
                tc::umma_commit(&sm.o_full);
            }
        }
    } else {
        // ------------------------------------------------------------ workers: gather, softmax, epilogue
        const uint32_t lane_addr = tbase + ((uint32_t)(warp * 32) << 16);
        const float scale_log2 = g.scale_log2;
        int bg = 0, blk = 0, n = 0, bg_n = 0, blk_n = 0, n_n = 0;
        uint32_t first = 0, first_n = 0;
        auto gather_issue = [&](int buf, int bgi, int ni) {
            const int b = bgi / g.Hkv, gk = bgi - b * g.Hkv;
            const size_t head0 = (size_t)(b * g.Hq + gk * g.G);
            for (int idx = tid; idx < ni * kChunks; idx += kGatherItemRows) {
                const int row = idx / kChunks, c = idx - row * kChunks;
                const uint32_t e = sm.ent[buf][row].x;
                const __nv_bfloat16* src = q_cube + ((head0 + ((e >> 21) & 15u)) * g.S_cap + (e & kEntryPosMask)) * D + c * 8;
                unsigned char* dst = reinterpret_cast<unsigned char*>(&sm.q[0][0][0]) + (c >> 3) * (128 * 128) + sw128(row, c & 7);
                cp_async_16(dst, src);
            }
            cp_async_commit();
        };
        item_col(0, bg, blk, first, n);
        if (tid < n) sm.ent[0][tid] = ws.entries[first + tid];
        // the workers meet on an mbarrier (bounded wait) once the entries of an item are in shared memory
        tc::mbar_arrive(&sm.ent_full);
        bool ok = tc::mbar_wait(&sm.ent_full, 0, abort_flag);
        if (ok) gather_issue(0, bg, n);
        for (int i = 0; ok && i < my_items; ++i) {
            const int cur = i & 1;
            cp_async_wait<0>();
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
            tc::mbar_arrive(&sm.q_full);
            const bool more = i + 1 < my_items;
            if (more) {
                item_col(i + 1, bg_n, blk_n, first_n, n_n);
                if (tid < n_n) sm.ent[cur ^ 1][tid] = ws.entries[first_n + tid];
                tc::mbar_arrive(&sm.ent_full);
            }
            const bool valid = tid < n;
            const uint2 ent = valid ? sm.ent[cur][tid] : make_uint2(0u, 0u);
            // ---- which of the 64 keys of the block this row attends: the cubes it selected, minus empty slots
            uint32_t m0 = 0u, m1 = 0u;
            if (valid) {
                const uint32_t sub = ent.x >> 25;
                if (g.c_shift >= 6) {
                    m0 = m1 = 0xffffffffu;
                } else if (g.c_shift == 5) {
                    m0 = (sub & 1u) ? 0xffffffffu : 0u;
                    m1 = (sub & 2u) ? 0xffffffffu : 0u;
                } else {
                    m0 = ((sub & 1u) ? 0x0000ffffu : 0u) | ((sub & 2u) ? 0xffff0000u : 0u);
                    m1 = ((sub & 4u) ? 0x0000ffffu : 0u) | ((sub & 8u) ? 0xffff0000u : 0u);
                }
                if (g.ragged) {
                    m0 &= __ldg(slot_valid + 2 * blk);
                    m1 &= __ldg(slot_valid + 2 * blk + 1);
                }
            }
            if (!(ok = tc::mbar_wait(&sm.s_full, i & 1, abort_flag))) break;
            tc::tc_fence_after_sync();
            uint32_t s[2][32];
            tc::tmem_ld_32x32(lane_addr, s[0]);
            tc::tmem_ld_32x32(lane_addr + 32, s[1]);
            tc::tmem_wait_ld();
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const uint32_t am = c ? m1 : m0;
                float a0 = -INFINITY, a1 = -INFINITY;
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    a0 = fmaxf(a0, ((am >> (2 * j)) & 1u) ? __uint_as_float(s[c][2 * j]) : -INFINITY);
                    a1 = fmaxf(a1, ((am >> (2 * j + 1)) & 1u) ? __uint_as_float(s[c][2 * j + 1]) : -INFINITY);
                }
                mx = fmax3(mx, a0, a1);
            }
            const float m_ref = mx * scale_log2;                   // -inf: no key of the block is visible to this row
            const float neg_ref = mx == -INFINITY ? 0.f : -m_ref;
            float l0 = 0.f, l1 = 0.f;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const uint32_t am = c ? m1 : m0;
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float p0 = fast_exp2(fmaf(__uint_as_float(s[c][2 * j]), scale_log2, ((am >> (2 * j)) & 1u) ? neg_ref : -INFINITY));
                    const float p1 = fast_exp2(fmaf(__uint_as_float(s[c][2 * j + 1]), scale_log2, ((am >> (2 * j + 1)) & 1u) ? neg_ref : -INFINITY));
                    l0 += p0;
                    l1 += p1;
                    pk[j] = pack_bf16x2(p0, p1);
                }
                tc::tmem_st_32x16(lane_addr + c * 16, pk);
            }
            const float l_sum = l0 + l1;
            tc::tmem_wait_st();
            tc::tc_fence_before_sync();
            tc::mbar_arrive(&sm.p_full);
            // ---- the S MMAs have completed: the Q tile can take the rows of the next item
            if (more) {
                if (!(ok = tc::mbar_wait(&sm.ent_full, (i + 1) & 1, abort_flag))) break;   // its entries are in shared memory
                gather_issue(cur ^ 1, bg_n, n_n);
            }
            // ---- epilogue: normalised partial output, (reference, sum)
            if (!(ok = tc::mbar_wait(&sm.o_full, i & 1, abort_flag))) break;
            tc::tc_fence_after_sync();
            const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
            uint4* dst = reinterpret_cast<uint4*>(ws.part_o + (size_t)ent.y * D);
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tc::tmem_ld_32x32(lane_addr + 64 + c * 32, o);
                tc::tmem_wait_ld();
                if (valid) {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint4 val;
                        val.x = pack_bf16x2(__uint_as_float(o[8 * q4 + 0]) * inv, __uint_as_float(o[8 * q4 + 1]) * inv);
                        val.y = pack_bf16x2(__uint_as_float(o[8 * q4 + 2]) * inv, __uint_as_float(o[8 * q4 + 3]) * inv);
                        val.z = pack_bf16x2(__uint_as_float(o[8 * q4 + 4]) * inv, __uint_as_float(o[8 * q4 + 5]) * inv);
                        val.w = pack_bf16x2(__uint_as_float(o[8 * q4 + 6]) * inv, __uint_as_float(o[8 * q4 + 7]) * inv);
                        dst[c * 4 + q4] = val;
                    }
                }
            }
            if (valid) ws.part_ml[ent.y] = make_float2(m_ref, l_sum);
            tc::tc_fence_before_sync();
            bg = bg_n; blk = blk_n; n = n_n; first = first_n;
        }
        cp_async_wait<0>();
    }
    // ---------------------------------------------------------------- teardown
    tc::tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
        if (sm.abort_flag) atomicExch(status, 6);   // a bounded wait expired
        else atomicAdd(executed_blocks, (unsigned long long)my_items);
    }
    if (warp == 4) tc::tmem_dealloc<kTmemCols>(tbase);
}

// ------------------------------------------------------------------------------------------------ merge
// D/8 threads per row, 16 bytes (8 elements) of the row each.
template <int D>
__global__ void __launch_bounds__(256) gather_merge_kernel(Geom g, GatherWs ws, __nv_bfloat16* __restrict__ out) {
    if (ws.ctrl[0] == 0u) return;
    constexpr int kLanes = D / 8, kRowsPerCta = 256 / kLanes;
    const int sub = threadIdx.x % kLanes;
    const int win = g.S - g.pos_begin;
    const long long n_rows = (long long)g.B * g.Hq * win;
    const unsigned gmask = kLanes == 32 ? 0xffffffffu : (((1u << kLanes) - 1u) << ((threadIdx.x & 31) / kLanes * kLanes));
    for (long long idx = (long long)blockIdx.x * kRowsPerCta + threadIdx.x / kLanes; idx < n_rows; idx += (long long)gridDim.x * kRowsPerCta) {
        const int bh = (int)(idx / win), pos = g.pos_begin + (int)(idx - (long long)bh * win);
        if (ws.pair_mode[(size_t)bh * ws.n_pairs_cap + pos / kPairRows] == 0u) continue;
        const size_t row = (size_t)bh * g.S_cap + pos;
        const uint32_t cnt = ws.row_cnt[row];
        if (cnt == 0u) continue;                                   // also every slot that holds no token
        const uint32_t ptr = ws.row_ptr[row];
        const float2 loc = ws.ml_local[row];
        float M = loc.x;
        for (uint32_t i = sub; i < cnt; i += kLanes) M = fmaxf(M, ws.part_ml[ptr + i].x);
#pragma unroll
        for (int d = 1; d < kLanes; d <<= 1) M = fmaxf(M, __shfl_xor_sync(gmask, M, d));
        const int b = bh / g.Hq, h = bh - b * g.Hq;
        uint4* dst = reinterpret_cast<uint4*>(out + (io_row(g, b, pos) * g.Hq + h) * D) + sub;
        float acc[8];
        float W = loc.y * exp2f(loc.x - M);
        {
            const uint4 v = *dst;
            const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[2 * k] = W * __uint_as_float(u[k] << 16);
                acc[2 * k + 1] = W * __uint_as_float(u[k] & 0xffff0000u);
            }
        }
        const uint4* src = reinterpret_cast<const uint4*>(ws.part_o + (size_t)ptr * D) + sub;
#pragma unroll 4
        for (uint32_t i = 0; i < cnt; ++i) {
            const float2 ml = ws.part_ml[ptr + i];
            const float w = ml.y * exp2f(ml.x - M);               // 0 for a partial without a visible key
            const uint4 v = __ldg(src + (size_t)i * kLanes);
            const uint32_t u[4] = {v.x, v.y, v.z, v.w};
            W += w;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[2 * k] = fmaf(w, __uint_as_float(u[k] << 16), acc[2 * k]);
                acc[2 * k + 1] = fmaf(w, __uint_as_float(u[k] & 0xffff0000u), acc[2 * k + 1]);
            }
        }
        const float inv = 1.f / W;
        uint4 res;
        res.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
        res.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
        res.z = pack_bf16x2(acc[4] * inv, acc[5] * inv);
        res.w = pack_bf16x2(acc[6] * inv, acc[7] * inv);
        *dst = res;
    }
}

}  // namespace adaspark
