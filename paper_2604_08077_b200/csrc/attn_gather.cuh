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
// Executed work = selected work, at the price of 2 D + 8 bytes written and read per entry (plus the gathered
// Q row).
//
// Which pairs of query tiles take this path is decided on the device, per pair, from the counts the selection
// left: entries of the pair's rows (P) against key blocks in the pair's union (U), gathered iff
// P <= pairs_per_block * U -- provided the qualifying pairs fit the workspace (else part of them, see
// kGatherClasses) and together save more than the path costs (kGatherMinGain).  The query rows are cut into a
// few row windows, and every (window, batch, kv head, key block) has its own entry list: the items of a window
// gather from a slice of Q that stays in L2.  Kernels, in launch order:
//   gather_count_kernel   per pair: row counts, P, U, the decision, entries per key block list (the warp's
//                         32 x 32 mask bits are transposed so that lane j holds the rows that selected cube j)
//   gather_scan_kernel    one CTA: which pairs are kept, prefix sums over pairs and key block lists
//   gather_items_kernel   work items of up to 128 entries of one list
//   (attn_prefill_tc_kernel, which reads the decisions)
//   gather_fill_kernel    per pair: row -> its slots, entries into the lists of their key blocks
//   attn_gather_kernel    per item: gathered Q rows x one key block -> partial results, in entry order
//   gather_merge_kernel   per row of the gathered pairs: merge into `out`
// The order of a list's entries depends on the order of atomics, but an entry's arithmetic does not depend
// on its neighbours in the item, and a row merges its partials in ascending block order: results are
// deterministic.
#pragma once
#include "attn_prefill_tc.cuh"

namespace adaspark {

constexpr int kGatherItemRows = 128;
constexpr int kGatherMaxWindows = 16;
constexpr int kGatherClasses = 4;       // a qualifying pair falls into a class by its ratio entries / union blocks:
                                        // <= 1/8, 1/4, 1/2 of the threshold, or up to the threshold.  When the
                                        // entries of all qualifying pairs exceed the workspace, (class, row window)
                                        // units are kept while they fit -- sparsest class first (its pairs gain most
                                        // per byte), inside a class the latest window first (longest unions) -- and
                                        // the other pairs stay on the union path; every unit counts its key blocks
                                        // in its own counters, so nothing is recounted
// Measured on a B200 (65536-token video, 1024 cubes): a (pair of tiles, key block) visit of the union kernel costs
// as much as about 44 entries of this path.  The path is taken only when the pairs that qualify save, by that
// estimate, at least kGatherMinGain entries' worth of time (~50 us): below that its fixed costs (six small
// launches, the scan) eat the gain.
constexpr long long kGatherBreakEven = 44;
constexpr long long kGatherMinGain = 300000;
constexpr uint32_t kEntryPosMask = 0x1fffffu;   // 21 bits of token index (a sequence holds at most 2^21 rows)

// Pointers into the forward workspace and sizes (all filled by the host).
struct GatherWs {
    uint32_t* ctrl;        // [0] entries, [1] items, [2] pairs on this path (0 entries: the path is off)
    uint32_t* pair_mode;   // [B*Hq*n_pairs_cap] 0: union path; c + 1: this path, ratio class c
    uint32_t* pair_cnt;    // entries of the pair's rows (0 when the pair stays on the tile kernel)
    uint32_t* pair_off;    // exclusive prefix sum of pair_cnt
    uint32_t* pair_u;      // key blocks in the pair's union (before its local range)
    uint32_t* pair_list;   // the pairs on this path, compacted (ctrl[2] of them)
    uint32_t* row_cnt;     // [B*Hq*S_cap] entries of a row
    uint32_t* row_ptr;     // index of the row's first slot in row_slots
    uint32_t* col_cnt;     // [kGatherClasses][lists * n_cols] entries of a key block list, per ratio class of the
                           // pairs they come from; zero at the start of a forward
    uint32_t* col_cur;     // [kGatherClasses][...] fill cursors; zero at the start of a forward
    uint32_t* col_roff;    // [kGatherClasses][...] first entry of the set's share of the block's list
    uint32_t* col_off;     // [lists * n_cols + 1] first entry of the block's list (exclusive prefix sum)
    uint32_t* col_item;    // [lists * n_cols + 1] first work item of the list
    uint4* items;          // (key block column, first entry, entries (<= 128), 0)
    uint32_t* entries;     // per key block, its entries: row of the call's tensors | head in group << 21 | cube bits << 25
    uint32_t* row_slots;   // per row (from row_ptr on), the indices of its entries in ascending block order
    __nv_bfloat16* part_o; // [cap_entries][D] normalised partial output of every entry (in entry order: an item
                           // of the attention kernel writes one contiguous piece)
    float2* part_ml;       // [cap_entries] (reference exponent in log2 units, sum)
    float2* ml_local;      // [B*Hq*S_cap] the same for the local range, written by the tile kernel
    uint32_t cap_entries;
    int n_cols;            // key blocks that hold video slots: ceil(S_v / 64)
    int n_lists;           // entry lists per key block column set: windows x B x Hkv (each of n_cols lists)
    int n_windows;         // row windows (<= kGatherMaxWindows)
    int pairs_per_window;  // The query rows are cut into windows of this many pairs of tiles and every (window,
                           // batch, kv head, key block) has its own entry list: the items of a window gather from a
                           // slice of Q that stays in L2, and a row's partial results lie close together.
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

// Transposes the 32 x 32 bit matrix whose row i is the word of lane i: afterwards bit i of lane j's word is the
// former bit j of lane i (five exchange steps on ever smaller blocks).  With rows = query rows and bits =
// cubes, lane j ends up with the set of rows that selected cube j: one step instead of one ballot per cube.
__device__ __forceinline__ uint32_t transpose_32x32(uint32_t x, int lane) {
    uint32_t y;
    y = __shfl_xor_sync(0xffffffffu, x, 16);
    x = (lane & 16) ? ((x & 0xffff0000u) | (y >> 16)) : ((x & 0x0000ffffu) | (y << 16));
    y = __shfl_xor_sync(0xffffffffu, x, 8);
    x = (lane & 8) ? ((x & 0xff00ff00u) | ((y >> 8) & 0x00ff00ffu)) : ((x & 0x00ff00ffu) | ((y << 8) & 0xff00ff00u));
    y = __shfl_xor_sync(0xffffffffu, x, 4);
    x = (lane & 4) ? ((x & 0xf0f0f0f0u) | ((y >> 4) & 0x0f0f0f0fu)) : ((x & 0x0f0f0f0fu) | ((y << 4) & 0xf0f0f0f0u));
    y = __shfl_xor_sync(0xffffffffu, x, 2);
    x = (lane & 2) ? ((x & 0xccccccccu) | ((y >> 2) & 0x33333333u)) : ((x & 0x33333333u) | ((y << 2) & 0xccccccccu));
    y = __shfl_xor_sync(0xffffffffu, x, 1);
    x = (lane & 1) ? ((x & 0xaaaaaaaau) | ((y >> 1) & 0x55555555u)) : ((x & 0x55555555u) | ((y << 1) & 0xaaaaaaaau));
    return x;
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

// entries of the lane's row before the pair's local range, in key blocks
__device__ __forceinline__ uint32_t row_entries(const Geom& g, const PairItem& it, const uint32_t* my) {
    const int bshift = max(g.c_shift - 6, 0);
    uint32_t cnt = 0;
#pragma unroll 4
    for (int w = 0; w < it.n_w; ++w) {
        uint32_t word = __ldg(my + (size_t)w * kTileRows);
        if (w == it.n_w - 1) word &= it.last_keep;
        cnt += (uint32_t)__popc(fold_to_blocks(word, g.c_shift)) << bshift;
    }
    return cnt;
}

// ------------------------------------------------------------------------------------------------ count
// One CTA per pair of query tiles and head.
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
    const uint32_t my_cnt = tile_ok ? row_entries(g, it, my) : 0u;
    uint32_t cnt = my_cnt;
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
        uint32_t mode = 0u;
        const float lim = ws.pairs_per_block * (float)U;
        if (P > 0 && (float)P <= lim) mode = (float)P <= 0.125f * lim ? 1u : ((float)P <= 0.25f * lim ? 2u : ((float)P <= 0.5f * lim ? 3u : 4u));
        const size_t slot = bh * ws.n_pairs_cap + it.pair;
        ws.pair_mode[slot] = mode;
        ws.pair_cnt[slot] = mode ? P : 0u;
        ws.pair_u[slot] = U;
        s_mode = mode;
    }
    __syncthreads();
    // rows of a pair that stays on the union path have no entries (the merge kernel reads only this)
    if (pos < g.S_cap) ws.row_cnt[bh * g.S_cap + pos] = s_mode ? my_cnt : 0u;
    if (!s_mode || !tile_ok) return;
    // entries per key block: the warp's 32 x 32 bits of a word are transposed, lane j then counts the rows that
    // selected cube 32 w + j and adds them to the cube's block(s)
    const int win = (it.pair - g.pos_begin / kPairRows) / ws.pairs_per_window;
    uint32_t* col_cnt = ws.col_cnt + ((size_t)(s_mode - 1u) * ws.n_lists + ((size_t)win * g.B + it.b) * g.Hkv + it.gk) * ws.n_cols;
    for (int w0 = 0; w0 < it.n_w; w0 += 4) {
        uint32_t wd[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) wd[k] = w0 + k < it.n_w ? __ldg(my + (size_t)(w0 + k) * kTileRows) : 0u;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (w0 + k >= it.n_w) break;
            if (w0 + k == it.n_w - 1) wd[k] &= it.last_keep;
            const uint32_t n = (uint32_t)__popc(transpose_32x32(fold_to_blocks(wd[k], g.c_shift), lane));
            if (n) {
                const int cube = (w0 + k) * 32 + lane;
                if (g.c_shift >= 6) {
                    for (int i = 0; i < (1 << bshift); ++i) atomicAdd(col_cnt + ((size_t)cube << bshift) + i, n);
                } else {
                    atomicAdd(col_cnt + (cube >> (6 - g.c_shift)), n);
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
    __shared__ uint32_t total_s, total_s2;
    const int tid = threadIdx.x;
    const int pair0 = g.pos_begin / kPairRows, n_pairs = (g.S + kPairRows - 1) / kPairRows - pair0;
    const int n_hb = g.Hq * g.B;
    const int n_slots = n_pairs * n_hb;
    // ---- which (ratio class, row window) units fit the workspace, and whether they are worth the fixed cost
    __shared__ unsigned long long unit_entries[kGatherClasses][kGatherMaxWindows];
    __shared__ long long unit_gain[kGatherClasses][kGatherMaxWindows];
    __shared__ uint32_t unit_keep[kGatherClasses];          // bit w: window w of the class takes the path
    __shared__ int any_keep_s;
    for (int i = tid; i < kGatherClasses * kGatherMaxWindows; i += 1024) {
        (&unit_entries[0][0])[i] = 0ull;
        (&unit_gain[0][0])[i] = 0ll;
    }
    __syncthreads();
    for (int idx = tid; idx < n_slots; idx += 1024) {
        const int hb = idx / n_pairs, pr = idx - hb * n_pairs;
        const size_t slot = (size_t)hb * ws.n_pairs_cap + pair0 + pr;
        const uint32_t mode = ws.pair_mode[slot];
        if (mode) {
            const uint32_t v = ws.pair_cnt[slot];
            const int win = pr / ws.pairs_per_window;
            atomicAdd(&unit_entries[mode - 1][win], (unsigned long long)v);
            atomicAdd(reinterpret_cast<unsigned long long*>(&unit_gain[mode - 1][win]),
                      (unsigned long long)(kGatherBreakEven * (long long)ws.pair_u[slot] - (long long)v));
        }
    }
    __syncthreads();
    if (tid == 0) {
        unsigned long long tot = 0ull;
        long long gain = 0ll;
        for (int c = 0; c < kGatherClasses; ++c) {
            uint32_t keep = 0u;
            for (int w = ws.n_windows - 1; w >= 0; --w) {
                const unsigned long long e = unit_entries[c][w];
                if (e == 0ull || tot + e > (unsigned long long)ws.cap_entries) continue;
                tot += e;
                gain += unit_gain[c][w];
                keep |= 1u << w;
            }
            unit_keep[c] = keep;
        }
        // (a threshold above the break-even estimate is a request to force the path: the estimate is not consulted)
        if (tot == 0ull || (ws.pairs_per_block <= (float)kGatherBreakEven && gain < kGatherMinGain)) {
            for (int c = 0; c < kGatherClasses; ++c) unit_keep[c] = 0u;
            tot = 0ull;
        }
        any_keep_s = tot != 0ull;
    }
    __syncthreads();
    const bool any_keep = any_keep_s != 0;
    // ---- pairs: offsets of their rows' partials, compact list; pairs of the other units go back to the union path
    unsigned long long carry = 0ull;
    uint32_t n_on = 0;
    for (int base = 0; base < n_slots; base += 1024) {
        const int idx = base + tid;
        size_t slot = 0;
        uint32_t v = 0;
        if (idx < n_slots) {
            const int hb = idx / n_pairs, pr = idx - hb * n_pairs;
            slot = (size_t)hb * ws.n_pairs_cap + pair0 + pr;
            const uint32_t mode = ws.pair_mode[slot];
            if (mode != 0u && ((unit_keep[mode - 1] >> (pr / ws.pairs_per_window)) & 1u)) v = ws.pair_cnt[slot];
            else if (mode != 0u) { ws.pair_mode[slot] = 0u; ws.pair_cnt[slot] = 0u; }
        }
        if (!any_keep) continue;
        const uint32_t ex = cta_exclusive_scan_1024(v, warp_sums, &total_s);
        if (idx < n_slots) ws.pair_off[slot] = (uint32_t)(carry + ex);
        const uint32_t exl = cta_exclusive_scan_1024(v != 0u ? 1u : 0u, warp_sums, &total_s2);
        if (idx < n_slots && v != 0u) ws.pair_list[n_on + exl] = (uint32_t)slot;
        n_on += total_s2;
        carry += total_s;
    }
    if (!any_keep) {
        // nothing to do, nothing fits, or too little to gain: every pair stays on the union path
        if (tid == 0) { ws.ctrl[0] = 0u; ws.ctrl[1] = 0u; ws.ctrl[2] = 0u; }
        return;
    }
    if (tid == 0) {
        ws.ctrl[0] = (uint32_t)carry;
        ws.ctrl[2] = n_on;
    }
    // ---- key blocks: offsets of their entry lists (and of every counter set's share) and of their work items.
    // Every thread owns a contiguous run of blocks: it sums them, one scan over the 1024 sums gives its start,
    // and it walks the run again (two scans in all instead of two per 1024 blocks).
    const int n_cols_all = ws.n_lists * ws.n_cols;
    const int cols_per_window = n_cols_all / ws.n_windows;       // lists are window-major
    const int per = (n_cols_all + 1023) / 1024;
    const int c0 = min(tid * per, n_cols_all), c1 = min(c0 + per, n_cols_all);
    uint32_t my_e = 0, my_i = 0;
    for (int col = c0; col < c1; ++col) {
        uint32_t v = 0;
        const int win = col / cols_per_window;
#pragma unroll
        for (int r = 0; r < kGatherClasses; ++r)
            if ((unit_keep[r] >> win) & 1u) v += ws.col_cnt[(size_t)r * n_cols_all + col];
        my_e += v;
        my_i += (v + kGatherItemRows - 1) / kGatherItemRows;
    }
    uint32_t e_off = cta_exclusive_scan_1024(my_e, warp_sums, &total_s);
    const uint32_t tot_e = total_s;
    uint32_t i_off = cta_exclusive_scan_1024(my_i, warp_sums, &total_s);
    const uint32_t tot_i = total_s;
    for (int col = c0; col < c1; ++col) {
        uint32_t o = e_off;
        ws.col_off[col] = o;
        ws.col_item[col] = i_off;
        uint32_t v = 0;
        const int win = col / cols_per_window;
#pragma unroll
        for (int r = 0; r < kGatherClasses; ++r) {
            if ((unit_keep[r] >> win) & 1u) {
                const uint32_t part = ws.col_cnt[(size_t)r * n_cols_all + col];
                ws.col_roff[(size_t)r * n_cols_all + col] = o;
                o += part;
                v += part;
            }
        }
        e_off += v;
        i_off += (v + kGatherItemRows - 1) / kGatherItemRows;
    }
    if (tid == 0) {
        ws.col_off[n_cols_all] = tot_e;
        ws.col_item[n_cols_all] = tot_i;
        ws.ctrl[1] = tot_i;
    }
}

// Work items of every key block: chunks of up to 128 entries of its list.  One warp per block.
__global__ void __launch_bounds__(256) gather_items_kernel(Geom g, GatherWs ws) {
    if (ws.ctrl[0] == 0u) return;
    const int n_cols_all = ws.n_lists * ws.n_cols;
    const int lane = threadIdx.x & 31;
    for (int col = blockIdx.x * 8 + (threadIdx.x >> 5); col < n_cols_all; col += gridDim.x * 8) {
        const uint32_t first = ws.col_off[col], n = ws.col_off[col + 1] - first, ib = ws.col_item[col];
        for (uint32_t c = lane; c * kGatherItemRows < n; c += 32)
            ws.items[ib + c] = make_uint4((uint32_t)col, first + c * kGatherItemRows, min(n - c * kGatherItemRows, (uint32_t)kGatherItemRows), 0u);
    }
}

// ------------------------------------------------------------------------------------------------ fill
__global__ void __launch_bounds__(256) gather_fill_kernel(Geom g, GatherWs ws, const uint32_t* __restrict__ tile_mask) {
    __shared__ uint32_t warp_tot[8];
    const PairItem it = pair_item(g, blockIdx.x);
    const size_t bh = (size_t)(it.b * g.Hq + it.h);
    const size_t slot = bh * ws.n_pairs_cap + it.pair;
    const uint32_t mode = ws.pair_mode[slot];
    if (ws.ctrl[0] == 0u || mode == 0u) return;
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
    const int win = (it.pair - g.pos_begin / kPairRows) / ws.pairs_per_window;
    const size_t colbase = ((size_t)(mode - 1u) * ws.n_lists + ((size_t)win * g.B + it.b) * g.Hkv + it.gk) * ws.n_cols;
    // an entry names its query row by the token's index in the call's tensors (what the gather needs), not by
    // its cube-major position: the conversion is done once here, not per copy in the attention kernel
    const uint32_t ent_x = (uint32_t)(slot_live(g, pos) ? pos_to_io(g, pos) - g.pos_begin : 0) | ((uint32_t)(it.h - it.gk * g.G) << 21);
    const uint32_t lt_mask = (1u << lane) - 1u;
    // Four words per step.  After the transposition lane j holds the rows of the warp that selected cube 32 w + j;
    // ONE round of atomics reserves the slots of all (word, cube) pairs of the step in their blocks' lists (the
    // return value of an atomic takes about a microsecond: one round per selected cube was the whole run time);
    // then every row walks its own cubes, fetching start and row set from the lane that owns the cube.
    const int group = g.c_shift >= 6 ? 1 : (kBlockTok >> g.c_shift);    // cubes per key block (small cubes)
    const int nblk = 1 << bshift;                                       // key blocks per cube (large cubes)
    for (int w0 = 0; w0 < it.n_w; w0 += 4) {
        uint32_t wd[4], fw[4], tw[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) wd[k] = w0 + k < it.n_w ? __ldg(my + (size_t)(w0 + k) * kTileRows) : 0u;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (w0 + k == it.n_w - 1) wd[k] &= it.last_keep;
            fw[k] = fold_to_blocks(wd[k], g.c_shift);
            tw[k] = transpose_32x32(fw[k], lane);
        }
        uint32_t slot0[4];                                              // first slot of the row for the cubes of word k
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            slot0[k] = ptr;
            ptr += (uint32_t)(__popc(fw[k]) * nblk);
        }
        for (int i = 0; i < nblk; ++i) {
            uint32_t st[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                st[k] = 0u;
                if (tw[k]) {
                    const int cube = (w0 + k) * 32 + lane;
                    const size_t col = colbase + (g.c_shift >= 6 ? ((size_t)cube << bshift) + i : (size_t)(cube >> (6 - g.c_shift)));
                    st[k] = ws.col_roff[col] + atomicAdd(ws.col_cur + col, (uint32_t)__popc(tw[k]));
                }
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                uint32_t t = fw[k];
                const int trips = __reduce_max_sync(0xffffffffu, __popc(t));
                for (int j = 0; j < trips; ++j) {
                    const int beta = t ? __ffs(t) - 1 : 0;
                    const uint32_t m = __shfl_sync(0xffffffffu, tw[k], beta), start = __shfl_sync(0xffffffffu, st[k], beta);
                    if (t) {
                        const uint32_t e = start + (uint32_t)__popc(m & lt_mask);
                        ws.entries[e] = ent_x | (((wd[k] >> beta) & ((1u << group) - 1u)) << 25);
                        ws.row_slots[slot0[k] + (uint32_t)(j * nblk + i)] = e;
                        t &= t - 1;
                    }
                }
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------ attention
// One persistent CTA per SM, 512 threads in four warpgroups:
//   warps 0-3 / 4-7   consumers of the even / odd items: softmax of S (thread = gathered row = TMEM lane),
//                     P into TMEM, normalised partial output and (reference, sum) to global memory
//   warps 8-11        gather producers: the Q rows of an item into a ring of three shared-memory tiles with
//                     cp.async (16 rows x 32 bytes per warp instruction), up to two items in flight
//   warp 12           MMA issuer: S_i = Q_i K^T (operands in shared memory), O_i = P_i V (P in TMEM); the S of
//                     item i+1 is issued before the P of item i is waited for, so the tensor pipe, the two
//                     softmax warpgroups and the gathers overlap
//   warp 13           TMA producer of the K / V^T blocks (ring of three)
//   warps 14-15       idle
// TMEM: consumer c owns columns [256 c, 256 c + 64) for S (P overwrites the first 32) and
// [256 c + 64, 256 c + 64 + D) for O.
constexpr int kGatherThreads = 512;
constexpr int kGatherRun = 16;          // consecutive items per CTA turn
constexpr int kGatherStages = 3;        // Q tiles in flight
constexpr int kGatherKvStages = 2;      // K / V^T tiles in flight
constexpr int kGatherOutPitch = 144;    // bytes per row of the output staging (128 + 16: conflict-free 16-byte accesses)

template <int D>
struct GatherSmem {
    __nv_bfloat16 q[kGatherStages][D / 64][128][64];   // [stage][d panel][gathered row][64 d], 128-byte swizzle
    __nv_bfloat16 k[kGatherKvStages][D / 64][64][64];  // [stage][d panel][key][64 d]
    __nv_bfloat16 v[kGatherKvStages][D][64];           // [stage][d][64 keys]  (V^T)
    unsigned char out_stage[8][32 * kGatherOutPitch];  // per consumer warp: 32 rows x 64 output columns (bf16)
    uint64_t q_full[kGatherStages], q_empty[kGatherStages], kv_full[kGatherKvStages], kv_empty[kGatherKvStages];
    uint64_t s_full[2], p_full[2], o_full[2];
    uint32_t tmem_base;
    int abort_flag;
};

template <int D>
__global__ void __launch_bounds__(kGatherThreads, 1) attn_gather_kernel(
    Geom g, GatherWs ws, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
    const __nv_bfloat16* __restrict__ q, const uint32_t* __restrict__ slot_valid,
    unsigned long long* __restrict__ executed_blocks, int32_t* __restrict__ status) {
    extern __shared__ unsigned char gather_smem_raw[];
    GatherSmem<D>& sm = *reinterpret_cast<GatherSmem<D>*>((reinterpret_cast<uintptr_t>(gather_smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kPanels = D / 64, kQKSteps = D / 16;
    constexpr uint32_t kIdescS = tc::make_idesc_bf16(128, 64);   // S: 128 gathered rows x 64 keys
    constexpr uint32_t kIdescO = tc::make_idesc_bf16(128, D);    // O: 128 rows x D
    constexpr uint32_t kKVBytes = 64 * D * 2 * 2;

    const uint32_t n_items = ws.ctrl[1];
    if (ws.ctrl[0] == 0u || (size_t)blockIdx.x * kGatherRun >= n_items) return;   // the path is off, or fewer runs than CTAs
    // Items are dealt to the CTAs in runs of kGatherRun: inside a run consecutive items mostly share their key
    // block, whose K / V^T tiles then stay in shared memory; across the grid all CTAs work on neighbouring runs,
    // i.e. on the same window of query rows, whose slice of Q stays in L2.
    const uint32_t n_runs = (n_items + kGatherRun - 1) / kGatherRun;
    const uint32_t my_runs = (n_runs - blockIdx.x + gridDim.x - 1) / gridDim.x;
    const bool has_tail = ((my_runs - 1) * gridDim.x + blockIdx.x) == n_runs - 1;   // the last (possibly short) run is this CTA's
    const int my_items = (int)(my_runs * kGatherRun - (has_tail ? n_runs * kGatherRun - n_items : 0u));
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    if (tid == 0) {
        for (int i = 0; i < kGatherStages; ++i) {
            tc::mbar_init(&sm.q_full[i], 128);
            tc::mbar_init(&sm.q_empty[i], 1);
        }
        for (int i = 0; i < kGatherKvStages; ++i) {
            tc::mbar_init(&sm.kv_full[i], 1);
            tc::mbar_init(&sm.kv_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            tc::mbar_init(&sm.s_full[i], 1);
            tc::mbar_init(&sm.p_full[i], 128);
            tc::mbar_init(&sm.o_full[i], 1);
        }
        sm.abort_flag = 0;
        tc::fence_barrier_init();
    }
    if (warp == 12) {
        tc::tmem_alloc<512>(&sm.tmem_base);
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
    // item i of this CTA: (column = ((window x batch) x kv head) * n_cols + key block, first entry, entries, -)
    auto item_at = [&](int i) -> uint4 {
        return __ldg(ws.items + ((size_t)(i / kGatherRun) * gridDim.x + blockIdx.x) * kGatherRun + (i % kGatherRun));
    };

    if (warp < 8) {
        // ------------------------------------------------------------ consumers
        const int c = warp >> 2, row = tid & 127;
        const uint32_t lane_addr = tbase + ((uint32_t)((warp & 3) * 32) << 16) + c * 256;
        const float scale_log2 = g.scale_log2;
        uint4 d_cur = c < my_items ? item_at(c) : make_uint4(0u, 0u, 0u, 0u);
        uint32_t ent = 0u;
        if (c < my_items && row < (int)d_cur.z) ent = __ldg(ws.entries + d_cur.y + row);
        for (int i = c, j = 0; i < my_items; i += 2, ++j) {
            // the next item of this warpgroup: descriptor and entry are requested now, used after the epilogue
            uint4 d_nxt = make_uint4(0u, 0u, 0u, 0u);
            if (i + 2 < my_items) d_nxt = item_at(i + 2);
            const bool valid = row < (int)d_cur.z;
            // ---- which of the 64 keys of the block this row attends: the cubes it selected, minus empty slots
            uint32_t m0 = 0u, m1 = 0u;
            if (valid) {
                const uint32_t sub = ent >> 25;
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
                    const int blk = (int)(d_cur.x % (uint32_t)ws.n_cols);
                    m0 &= __ldg(slot_valid + 2 * blk);
                    m1 &= __ldg(slot_valid + 2 * blk + 1);
                }
            }
            if (!tc::mbar_wait(&sm.s_full[c], j & 1, abort_flag)) break;
            tc::tc_fence_after_sync();
            uint32_t s[2][32];
            tc::tmem_ld_32x32(lane_addr, s[0]);
            tc::tmem_ld_32x32(lane_addr + 32, s[1]);
            tc::tmem_wait_ld();
            const bool full = (m0 & m1) == 0xffffffffu;
            float mx = -INFINITY;
            if (full) {
                float a[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    a[0] = fmax3(a[0], __uint_as_float(s[0][4 * t]), __uint_as_float(s[0][4 * t + 1]));
                    a[1] = fmax3(a[1], __uint_as_float(s[0][4 * t + 2]), __uint_as_float(s[0][4 * t + 3]));
                    a[2] = fmax3(a[2], __uint_as_float(s[1][4 * t]), __uint_as_float(s[1][4 * t + 1]));
                    a[3] = fmax3(a[3], __uint_as_float(s[1][4 * t + 2]), __uint_as_float(s[1][4 * t + 3]));
                }
                mx = fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3]));
            } else {
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    const uint32_t am = hf ? m1 : m0;
                    float a0 = -INFINITY, a1 = -INFINITY;
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        a0 = fmaxf(a0, ((am >> (2 * t)) & 1u) ? __uint_as_float(s[hf][2 * t]) : -INFINITY);
                        a1 = fmaxf(a1, ((am >> (2 * t + 1)) & 1u) ? __uint_as_float(s[hf][2 * t + 1]) : -INFINITY);
                    }
                    mx = fmax3(mx, a0, a1);
                }
            }
            const float m_ref = mx * scale_log2;                   // -inf: no key of the block is visible to this row
            const float neg_ref = mx == -INFINITY ? 0.f : -m_ref;
            float l0 = 0.f, l1 = 0.f;
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const uint32_t am = hf ? m1 : m0;
                uint32_t pk[16];
                if (full) {
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(s[hf][2 * t]), scale_log2, neg_ref));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(s[hf][2 * t + 1]), scale_log2, neg_ref));
                        l0 += p0;
                        l1 += p1;
                        pk[t] = pack_bf16x2(p0, p1);
                    }
                } else {
#pragma unroll
                    for (int t = 0; t < 16; ++t) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(s[hf][2 * t]), scale_log2, ((am >> (2 * t)) & 1u) ? neg_ref : -INFINITY));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(s[hf][2 * t + 1]), scale_log2, ((am >> (2 * t + 1)) & 1u) ? neg_ref : -INFINITY));
                        l0 += p0;
                        l1 += p1;
                        pk[t] = pack_bf16x2(p0, p1);
                    }
                }
                tc::tmem_st_32x16(lane_addr + hf * 16, pk);
            }
            const float l_sum = l0 + l1;
            tc::tmem_wait_st();
            tc::tc_fence_before_sync();
            tc::mbar_arrive(&sm.p_full[c]);
            uint32_t e_nxt = 0u;
            if (i + 2 < my_items && row < (int)d_nxt.z) e_nxt = __ldg(ws.entries + d_nxt.y + row);
            // ---- epilogue: normalised partial output, (reference, sum)
            if (!tc::mbar_wait(&sm.o_full[c], j & 1, abort_flag)) break;
            tc::tc_fence_after_sync();
            const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
            // The output rows in rounds of 64 columns.  A thread holds one row, but 32 threads storing 16 bytes to 32
            // different rows cost the L1 one step per row; so the warp transposes through shared memory and writes its
            // 32 rows (contiguous in the partial buffer: entry order) as whole 128-byte lines, four rows per
            // instruction.
            unsigned char* stage = sm.out_stage[warp];
            unsigned char* gdst = reinterpret_cast<unsigned char*>(ws.part_o + (size_t)(d_cur.y + (row & ~31)) * D);
            const int n_warp_rows = min(32, (int)d_cur.z - (row & ~31));          // rows of this warp that hold an entry
#pragma unroll
            for (int hf = 0; hf < D / 64; ++hf) {
                uint32_t o[2][32];
                tc::tmem_ld_32x32(lane_addr + 64 + hf * 64, o[0]);
                tc::tmem_ld_32x32(lane_addr + 64 + hf * 64 + 32, o[1]);
                tc::tmem_wait_ld();
#pragma unroll
                for (int cc = 0; cc < 2; ++cc) {
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint4 val;
                        val.x = pack_bf16x2(__uint_as_float(o[cc][8 * q4 + 0]) * inv, __uint_as_float(o[cc][8 * q4 + 1]) * inv);
                        val.y = pack_bf16x2(__uint_as_float(o[cc][8 * q4 + 2]) * inv, __uint_as_float(o[cc][8 * q4 + 3]) * inv);
                        val.z = pack_bf16x2(__uint_as_float(o[cc][8 * q4 + 4]) * inv, __uint_as_float(o[cc][8 * q4 + 5]) * inv);
                        val.w = pack_bf16x2(__uint_as_float(o[cc][8 * q4 + 6]) * inv, __uint_as_float(o[cc][8 * q4 + 7]) * inv);
                        *reinterpret_cast<uint4*>(stage + lane * kGatherOutPitch + (cc * 4 + q4) * 16) = val;
                    }
                }
                __syncwarp();
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int r = j * 4 + (lane >> 3), ch = lane & 7;
                    const uint4 val = *reinterpret_cast<const uint4*>(stage + r * kGatherOutPitch + ch * 16);
                    if (r < n_warp_rows) __stcs(reinterpret_cast<uint4*>(gdst + (size_t)r * (2 * D) + hf * 128 + ch * 16), val);   // written once, read once: keep it from displacing Q in L2
                }
                __syncwarp();
            }
            tc::tc_fence_before_sync();
            if (valid) {
                __stcs(ws.part_ml + d_cur.y + row, make_float2(m_ref, l_sum));
            }
            d_cur = d_nxt;
            ent = e_nxt;
        }
    } else if (warp < 12) {
        // ------------------------------------------------------------ gather producers
        // A row of Q is 2 D bytes = 2 D / 16 pieces of 16 bytes; consecutive lanes copy consecutive pieces, so a warp
        // instruction covers whole 128-byte lines of one or two rows (16 rows x 32 bytes per instruction cost the L1 one
        // step per row and made this kernel L1-bound).  The warpgroup copies 128 / kRowsPerPass rows per pass.
        constexpr int kPieces = D / 8;                               // 16-byte pieces per row
        constexpr int kRowsPerPass = 128 / kPieces;                  // rows the 128 producer threads cover per pass
        const int pt = tid - 256;                                  // 0..127
        const int piece = pt % kPieces, rsub = pt / kPieces;
        constexpr int kPasses = 128 / kRowsPerPass;
        uint4 d_cur = item_at(0);
        // the entries of the next item are requested while the rows of this one are copied: a load of the entry
        // right before its copy left this warpgroup waiting on L2 latency once per pass
        uint32_t e_cur[kPasses], e_nxt[kPasses];
#pragma unroll
        for (int ps = 0; ps < kPasses; ++ps) e_cur[ps] = (ps * kRowsPerPass + rsub < (int)d_cur.z) ? __ldg(ws.entries + d_cur.y + ps * kRowsPerPass + rsub) : 0u;
        bool ok = true;
        for (int i = 0; i < my_items; ++i) {
            const int st = i % kGatherStages;
            uint4 d_nxt = make_uint4(0u, 0u, 0u, 0u);
            if (i + 1 < my_items) d_nxt = item_at(i + 1);
            const int n = (int)d_cur.z;
#pragma unroll
            for (int ps = 0; ps < kPasses; ++ps) e_nxt[ps] = (ps * kRowsPerPass + rsub < (int)d_nxt.z) ? __ldg(ws.entries + d_nxt.y + ps * kRowsPerPass + rsub) : 0u;
            if (!(ok = tc::mbar_wait(&sm.q_empty[st], ((i / kGatherStages) & 1) ^ 1, abort_flag))) break;
            const int bg = (int)(d_cur.x / (uint32_t)ws.n_cols) % (g.B * g.Hkv);
            const int b = bg / g.Hkv, gk = bg - b * g.Hkv;
            const int head0 = gk * g.G;
            unsigned char* qbase = reinterpret_cast<unsigned char*>(&sm.q[st][0][0][0]) + (piece >> 3) * (128 * 128);
#pragma unroll
            for (int ps = 0; ps < kPasses; ++ps) {
                const int row = ps * kRowsPerPass + rsub;
                if (row < n) {
                    const uint32_t e = e_cur[ps];
                    // the row's place in the caller's tensor [B, S_io, Hq, D]
                    const __nv_bfloat16* src = q + (((size_t)b * g.S_io + (e & kEntryPosMask)) * g.Hq + head0 + (int)((e >> 21) & 15u)) * D;
                    cp_async_16(qbase + sw128(row, piece & 7), src + piece * 8);
                }
            }
#pragma unroll
            for (int ps = 0; ps < kPasses; ++ps) e_cur[ps] = e_nxt[ps];
            cp_async_commit();
            if (i > 0) {                                             // the previous item has landed
                cp_async_wait<1>();
                asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
                tc::mbar_arrive(&sm.q_full[(i - 1) % kGatherStages]);
            }
            d_cur = d_nxt;
        }
        cp_async_wait<0>();
        if (ok) {
            asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
            tc::mbar_arrive(&sm.q_full[(my_items - 1) % kGatherStages]);
        }
    } else if (warp == 12) {
        // ------------------------------------------------------------ MMA issuer (one thread)
        if (lane == 0) {
            constexpr uint32_t kQPanelStep = (128 * 64 * 2) >> 4, kKPanelStep = (64 * 64 * 2) >> 4, kKStep = 32 >> 4;
            // K / V^T stage of an item: a new one only when the key block changes (kvn counts the loads so far)
            int kvn_s = -1, kvn_pv = -1;
            uint32_t col_s = 0xffffffffu, col_pv = 0xffffffffu;
            auto issue_s = [&](int i) -> bool {
                const int st = i % kGatherStages, ph = (i / kGatherStages) & 1;
                const uint32_t col = item_at(i).x;
                if (col != col_s) { col_s = col; ++kvn_s; }
                const int kst = kvn_s % kGatherKvStages;
                if (!tc::mbar_wait(&sm.q_full[st], ph, abort_flag)) return false;
                if (!tc::mbar_wait(&sm.kv_full[kst], (kvn_s / kGatherKvStages) & 1, abort_flag)) return false;
                tc::tc_fence_after_sync();
                const uint32_t q_lo = tc::smem_desc_lo_sw128(smem_u32(&sm.q[st][0][0][0]));
                const uint32_t k_lo = tc::smem_desc_lo_sw128(smem_u32(&sm.k[kst][0][0][0]));
                const uint32_t dst = tbase + (i & 1) * 256;
#pragma unroll
                for (int ks = 0; ks < kQKSteps; ++ks) {
                    const uint32_t qo = (ks >> 2) * kQPanelStep + (ks & 3) * kKStep, ko = (ks >> 2) * kKPanelStep + (ks & 3) * kKStep;
                    tc::umma_ss(dst, tc::smem_desc_from_halves(q_lo + qo, tc::kSmemDescHiSw128),
                                tc::smem_desc_from_halves(k_lo + ko, tc::kSmemDescHiSw128), kIdescS, ks > 0);
                }
                tc::umma_commit(&sm.s_full[i & 1]);
                tc::umma_commit(&sm.q_empty[st]);                      // the Q tile is free once these MMAs have run
                return true;
            };
            bool ok = issue_s(0);
            for (int i = 0; ok && i < my_items; ++i) {
                // S of the next item (other TMEM set; its P of two items ago was consumed by an earlier MMA of this thread)
                if (i + 1 < my_items && !(ok = issue_s(i + 1))) break;
                if (!(ok = tc::mbar_wait(&sm.p_full[i & 1], (i >> 1) & 1, abort_flag))) break;
                tc::tc_fence_after_sync();
                const uint32_t col = item_at(i).x;
                if (col != col_pv) { col_pv = col; ++kvn_pv; }
                const int kst = kvn_pv % kGatherKvStages;
                const uint32_t v_lo = tc::smem_desc_lo_sw128(smem_u32(&sm.v[kst][0][0]));
                const uint32_t set = tbase + (i & 1) * 256;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    tc::umma_ts(set + 64, set + ks * 8, tc::smem_desc_from_halves(v_lo + ks * kKStep, tc::kSmemDescHiSw128), kIdescO, ks > 0);
                tc::umma_commit(&sm.o_full[i & 1]);
                // the stage is free after the last item of its key block
                if (i + 1 == my_items || item_at(i + 1).x != col) tc::umma_commit(&sm.kv_empty[kst]);
            }
        }
    } else if (warp == 13) {
        // ------------------------------------------------------------ TMA producer of K / V^T blocks
        if (lane == 0) {
            int kvn = -1;
            uint32_t col_prev = 0xffffffffu;
            for (int i = 0; i < my_items; ++i) {
                const uint32_t col = item_at(i).x;
                if (col == col_prev) continue;                         // same key block as the item before: tiles stay
                col_prev = col;
                ++kvn;
                const int st = kvn % kGatherKvStages;
                const int list = (int)(col / (uint32_t)ws.n_cols), blk = (int)(col - (uint32_t)list * (uint32_t)ws.n_cols);
                const int bg = list % (g.B * g.Hkv);
                if (!tc::mbar_wait(&sm.kv_empty[st], ((kvn / kGatherKvStages) & 1) ^ 1, abort_flag)) break;
                tc::mbar_arrive_expect_tx(&sm.kv_full[st], kKVBytes);
                for (int p = 0; p < kPanels; ++p)
                    tc::tma_load_2d(&sm.k[st][p][0][0], &tmK, p * 64, bg * g.S_cap + blk * kBlockTok, &sm.kv_full[st]);
                tc::tma_load_2d(&sm.v[st][0][0], &tmV, 0, (bg * g.n_kv_blocks_cap + blk) * D, &sm.kv_full[st]);
            }
        }
    }
    // ---------------------------------------------------------------- teardown
    tc::tc_fence_before_sync();
    __syncthreads();
    if (tid == 0) {
        if (sm.abort_flag) atomicExch(status, 6);   // a bounded wait expired
        else atomicAdd(executed_blocks, (unsigned long long)my_items);
    }
    if (warp == 12) tc::tmem_dealloc<512>(tbase);
}

// ------------------------------------------------------------------------------------------------ merge
// D/8 threads per row, 16 bytes (8 elements) of the row each.  The partials are folded in one pass with a
// running reference exponent (their loads do not depend on it, so several are in flight per thread).
template <int D>
__global__ void __launch_bounds__(256) gather_merge_kernel(Geom g, GatherWs ws, __nv_bfloat16* __restrict__ out) {
    if (ws.ctrl[0] == 0u) return;
    constexpr int kLanes = D / 8, kRowsPerCta = 256 / kLanes;
    const int sub = threadIdx.x % kLanes;
    const long long n_rows = (long long)ws.ctrl[2] * kPairRows;    // the rows of the pairs on this path
    for (long long idx = (long long)blockIdx.x * kRowsPerCta + threadIdx.x / kLanes; idx < n_rows; idx += (long long)gridDim.x * kRowsPerCta) {
        const uint32_t slot = __ldg(ws.pair_list + (idx >> 8));
        const int bh = (int)(slot / (uint32_t)ws.n_pairs_cap);
        const int pos = (int)(slot - (uint32_t)bh * (uint32_t)ws.n_pairs_cap) * kPairRows + (int)(idx & 255);
        if (pos >= g.S) continue;
        const size_t row = (size_t)bh * g.S_cap + pos;
        // everything that does not depend on the row's count is requested first (one round of memory latency)
        const uint32_t cnt = __ldg(ws.row_cnt + row);              // 0: a pair on the union path, or a slot without token
        const uint32_t ptr = __ldg(ws.row_ptr + row);
        const float2 loc = __ldg(ws.ml_local + row);
        if (cnt == 0u) continue;
        const int b = bh / g.Hq, h = bh - b * g.Hq;
        uint4* dst = reinterpret_cast<uint4*>(out + (io_row(g, b, pos) * g.Hq + h) * D) + sub;
        const uint4 own = *dst;
        const uint4* src = reinterpret_cast<const uint4*>(ws.part_o) + sub;
        float acc[8];
        float M = loc.x, W = loc.y;                                // the local range always has a visible key
        {
            const uint32_t u[4] = {own.x, own.y, own.z, own.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                acc[2 * k] = W * __uint_as_float(u[k] << 16);
                acc[2 * k + 1] = W * __uint_as_float(u[k] & 0xffff0000u);
            }
        }
        for (uint32_t i0 = 0; i0 < cnt; i0 += 4) {
            // four partials at a time: indices, then (m, l) and data of all four, then the arithmetic
            uint32_t e[4];
            float2 ml[4];
            uint4 v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) e[k] = i0 + k < cnt ? __ldg(ws.row_slots + ptr + i0 + k) : 0xffffffffu;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                ml[k] = make_float2(0.f, 0.f);
                v[k] = make_uint4(0u, 0u, 0u, 0u);
                if (e[k] != 0xffffffffu) {
                    ml[k] = __ldcs(ws.part_ml + e[k]);
                    v[k] = __ldcs(src + (size_t)e[k] * kLanes);
                }
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                if (ml[k].y > 0.f) {                               // a partial without a visible key has sum 0
                    const uint32_t u[4] = {v[k].x, v[k].y, v[k].z, v[k].w};
                    const float Mn = fmaxf(M, ml[k].x);
                    const float so = exp2f(M - Mn), w = ml[k].y * exp2f(ml[k].x - Mn);
                    M = Mn;
                    W = fmaf(W, so, w);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        acc[2 * q] = fmaf(w, __uint_as_float(u[q] << 16), acc[2 * q] * so);
                        acc[2 * q + 1] = fmaf(w, __uint_as_float(u[q] & 0xffff0000u), acc[2 * q + 1] * so);
                    }
                }
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
