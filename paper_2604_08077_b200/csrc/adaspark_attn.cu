// C-ABI entry points of libadaspark_attn: host-side validation, workspace carving and kernel
// launches.  All arithmetic lives in the kernels included below; see include/adaspark_attn.h for
// the contract of every call.
#include "../../include/adaspark_attn.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>

#include "common.cuh"
#include "relayout_pool.cuh"
#include "select_exact.cuh"
#include "attn_prefill_mma.cuh"
#include "tc_common.cuh"
#include "decode.cuh"
#include "decode_splitkv.cuh"
#ifdef ADASPARK_WITH_TCGEN05
#include "attn_prefill_tc.cuh"
#include "score_select_fused.cuh"
#include "attn_gather.cuh"
#endif

using namespace adaspark;

struct adaspark_attn {
    adaspark_attn_config_t cfg;
    bool partitioned;
    int B, T, H, W, n_text_max;
    int C, N, S_v, S_cap;
    adaspark_attn_layout_t layout;
    // workspace carving (byte offsets)
    size_t fw_status_off, fw_headmax_off, fw_valid_off, fw_gcol_off, fw_mask_off, fw_union_off, fw_fallback_off, fw_scratch_off,
        fw_kplanes_off, fw_gpair_off, fw_grow_off, fw_gml_off, fw_gitems_off, fw_gentries_off, fw_gparto_off,
        fw_gpartml_off, fw_total;
    // query-gather path of the prefill: capacity in (row, key block) entries, decision threshold, byte budget
    uint32_t gather_cap;
    int gather_windows;
    float gather_pairs_per_block;
    uint64_t gather_budget;
    size_t dc_status_off, dc_bitmap_off, dc_items_off, dc_nitems_off, dc_partial_off, dc_total;
    int dc_splits;
    int prefill_kernel;
    int sm_count;
    int64_t launches;
    bool timing;
    cudaEvent_t ev[7];          // stage boundaries [0..4], around the union attention kernel of the prefill [5, 6]
    bool ev_recorded;
    char err[256];
};

namespace {

constexpr size_t kAlign = 256;
constexpr int kExactCtas = 296;   // CTAs of the fp64 selection kernel (its scratch rows are sized for them)
// query-gather path: pairs of query tiles take it when their rows' (row, key block) entries are at most this
// many per key block of the pair's union (measured break-even on a B200, see the attention profile), and the
// partial results of all such pairs must fit this many bytes of workspace
constexpr float kGatherDefaultPairsPerBlock = 30.f;
constexpr uint64_t kGatherDefaultBudget = 24ull << 30;
constexpr uint64_t kGatherEntriesPerRow = 128;
constexpr size_t kGatherWindowBytes = 40u << 20;
size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }

adaspark_status_t fail(adaspark_attn* h, adaspark_status_t st, const char* fmt, ...) {
    if (h) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(h->err, sizeof(h->err), fmt, ap);
        va_end(ap);
    }
    return st;
}

// Geometry of one call.  frame_begin / frame_end delimit the video frames this call brings (whole time
// blocks of cubes); n_text text tokens are present after the call (0 while the video is incomplete).
Geom make_geom(const adaspark_attn* h, int n_text, int frame_begin = 0, int frame_end = -1, int n_prefix = 0) {
    Geom g;
    if (frame_end < 0) frame_end = h->T;
    g.B = h->B; g.T = h->T; g.H = h->H; g.W = h->W;
    g.ct = h->cfg.cube_t; g.ch = h->cfg.cube_h; g.cw = h->cfg.cube_w;
    g.nH = (h->H + g.ch - 1) / g.ch; g.nW = (h->W + g.cw - 1) / g.cw;
    g.ragged = (h->T % g.ct || h->H % g.ch || h->W % g.cw) ? 1 : 0;
    g.S_tok = h->T * h->H * h->W;
    g.n_prefix = n_prefix;
    g.C = h->C; g.N = h->N;
    g.c_shift = 0;
    while ((1 << g.c_shift) < g.C) ++g.c_shift;
    g.cw_shift = 0;
    while ((1 << g.cw_shift) < g.cw) ++g.cw_shift;
    g.ch_shift = 0;
    while ((1 << g.ch_shift) < g.ch) ++g.ch_shift;
    g.S_v = h->S_v; g.n_text = n_text + n_prefix;
    // slots present after the call (text only once the video is complete; chunks need H and W divisible,
    // so that frames count the same in tokens and in slots)
    g.S = (frame_end == h->T ? h->S_v : frame_end * h->H * h->W) + n_prefix + n_text;
    g.pos_begin = frame_begin * h->H * h->W;
    g.frame_begin = frame_begin;
    g.S_io = (frame_end - frame_begin) * h->H * h->W + n_prefix + n_text;
    g.tile_begin = g.pos_begin / kTileRows;
    g.N_live = ((frame_end + g.ct - 1) / g.ct) * g.nH * g.nW;
    g.S_cap = h->S_cap;
    g.n_words = (h->N + 31) / 32;
    g.n_tiles = (g.S + kTileRows - 1) / kTileRows;
    g.n_tiles_cap = h->S_cap / kTileRows;
    g.div_nW.init(g.nW);
    g.div_nH.init(g.nH);
    g.div_n_tiles.init(g.n_tiles);
    g.n_kv_blocks_cap = h->S_cap / kBlockTok;
    g.Hq = h->cfg.n_q_heads; g.Hkv = h->cfg.n_kv_heads; g.G = g.Hq / g.Hkv; g.D = h->cfg.head_dim;
    g.div_Hq.init(g.Hq);
    g.N_ld = (h->N + 63) / 64 * 64;
    double scale = h->cfg.softmax_scale > 0.f ? (double)h->cfg.softmax_scale : 1.0 / std::sqrt((double)g.D);
    g.scale_d = scale;
    g.scale = (float)scale;
    g.scale_log2 = (float)(scale * 1.4426950408889634);
    g.top_p = (double)h->cfg.top_p;
    g.top_k = h->cfg.top_k;
    return g;
}

void mark(adaspark_attn* h, int i, cudaStream_t st) {
    if (h->timing) {
        cudaEventRecord(h->ev[i], st);
        h->ev_recorded = true;
    }
}

bool launch_ok(adaspark_attn* h, const char* what) {
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        fail(h, ADASPARK_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
        return false;
    }
    h->launches++;
    return true;
}

template <typename K>
bool set_smem(adaspark_attn* h, K kernel, size_t bytes, const char* what) {
    if (bytes <= 48 * 1024) return true;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
    if (e != cudaSuccess) {
        fail(h, ADASPARK_ERR_CUDA, "%s: cudaFuncSetAttribute(%zu): %s", what, bytes, cudaGetErrorString(e));
        return false;
    }
    return true;
}

}  // namespace

extern "C" {

adaspark_status_t adaspark_attn_create(const adaspark_attn_config_t* config, adaspark_attn_t** out_handle) {
    if (!config || !out_handle) return ADASPARK_ERR_INVALID_ARG;
    *out_handle = nullptr;
    if (config->cube_t <= 0 || config->cube_h <= 0 || config->cube_w <= 0 || config->n_q_heads <= 0 ||
        config->n_kv_heads <= 0 || config->head_dim <= 0 || !(config->top_p > 0.f) ||
        config->softmax_scale < 0.f || config->device < 0 || config->top_k < 0)
        return ADASPARK_ERR_INVALID_ARG;
    if (config->n_q_heads % config->n_kv_heads != 0) return ADASPARK_ERR_INVALID_ARG;
    if (config->head_dim != 64 && config->head_dim != 128) return ADASPARK_ERR_UNSUPPORTED;
    if (config->n_q_heads / config->n_kv_heads > 16) return ADASPARK_ERR_UNSUPPORTED;
    long long C = (long long)config->cube_t * config->cube_h * config->cube_w;
    if (C != 16 && C != 32 && C != 64 && C != 128 && C != 256 && C != 512 && C != 1024) return ADASPARK_ERR_UNSUPPORTED;
    adaspark_attn* h = new (std::nothrow) adaspark_attn();
    if (!h) return ADASPARK_ERR_INVALID_ARG;
    std::memset(h, 0, sizeof(*h));
    h->cfg = *config;
    h->C = (int)C;
#ifdef ADASPARK_WITH_TCGEN05
    h->prefill_kernel = 1;
    h->gather_pairs_per_block = kGatherDefaultPairsPerBlock;
    h->gather_budget = kGatherDefaultBudget;
#else
    h->prefill_kernel = 0;
#endif
    *out_handle = h;
    return ADASPARK_OK;
}

adaspark_status_t adaspark_attn_partition(adaspark_attn_t* h, int32_t batch, int32_t frames, int32_t grid_h,
                                          int32_t grid_w, int32_t n_text_max, size_t* workspace_bytes) {
    if (!h) return ADASPARK_ERR_INVALID_ARG;
    if (batch <= 0 || frames <= 0 || grid_h <= 0 || grid_w <= 0 || n_text_max < 0)
        return fail(h, ADASPARK_ERR_INVALID_ARG, "partition: non-positive size");
    const adaspark_attn_config_t& c = h->cfg;
    // a grid the window does not divide is covered by ceil() cubes per axis; the far cubes hold fewer tokens
    long long N = (long long)((frames + c.cube_t - 1) / c.cube_t) * ((grid_h + c.cube_h - 1) / c.cube_h) *
                  ((grid_w + c.cube_w - 1) / c.cube_w);
    if (N > 4096) return fail(h, ADASPARK_ERR_UNSUPPORTED, "partition: %lld cubes > 4096", N);
    long long S_v = N * h->C;                                // cache slots of the video (= tokens unless ragged)
    long long S_cap = (S_v + n_text_max + 1 + 127) / 128 * 128;
    if ((long long)batch * S_cap * c.n_q_heads * c.head_dim >= (1ll << 40) || S_cap >= (1ll << 30))
        return fail(h, ADASPARK_ERR_UNSUPPORTED, "partition: problem too large");
#ifdef ADASPARK_WITH_TCGEN05
    // the attention kernel keeps one bit per 64-key block of a sequence in shared memory
    if (S_cap / kBlockTok > 32ll * kMaxBlockWords)
        return fail(h, ADASPARK_ERR_UNSUPPORTED, "partition: %lld cache rows per sequence > %d", S_cap,
                    32 * kMaxBlockWords * kBlockTok);
#endif
    h->B = batch; h->T = frames; h->H = grid_h; h->W = grid_w; h->n_text_max = n_text_max;
    h->N = (int)N; h->S_v = (int)S_v; h->S_cap = (int)S_cap;

    const int D = c.head_dim, Hq = c.n_q_heads, Hkv = c.n_kv_heads;
    const size_t n_words = (size_t)(N + 31) / 32, N_ld = (size_t)(N + 63) / 64 * 64;
    const size_t n_tiles_cap = (size_t)S_cap / kTileRows;
    adaspark_attn_layout_t& L = h->layout;
    L.n_cubes = N; L.cube_tokens = h->C; L.s_video = S_v; L.s_cap = S_cap; L.bitmap_words = (int64_t)n_words;
    L.k_cube_bytes = (int64_t)((size_t)batch * Hkv * S_cap * D * 2);
    L.v_cube_bytes = L.k_cube_bytes;
    L.cube_keys_bytes = (int64_t)((size_t)batch * Hkv * N * D * 4);

    // forward workspace: header | head exponents | per-tile mask matrix | per-tile union words | rows left to
    // the fp64 selection kernel | its score scratch | key digit planes (tcgen05 path)
    size_t off = 0;
    h->fw_status_off = off; off = align_up(off + 256);
    h->fw_headmax_off = off; off = align_up(off + (size_t)batch * Hkv * 4 * 2);   // key exponents, then largest |k|^2
    h->fw_valid_off = off; off = align_up(off + (size_t)(S_cap / kBlockTok) * 2 * 4);   // which slots of a block hold a token
    const size_t n_cols = (size_t)(S_v + kBlockTok - 1) / kBlockTok;                     // key blocks that hold video
    // query-gather path: the rows are cut into windows whose slice of Q (all heads) is about a third of the L2
    {
        const size_t q_bytes = (size_t)batch * Hq * S_cap * D * 2;
        size_t w = (q_bytes + kGatherWindowBytes - 1) / kGatherWindowBytes;
        h->gather_windows = (int)(w < 1 ? 1 : (w > 16 ? 16 : w));
    }
    const size_t n_lists = (size_t)h->gather_windows * batch * Hkv;
    h->fw_gcol_off = off; off = align_up(off + n_lists * n_cols * 2 * kGatherClasses * 4);   // entry counts and fill cursors (zeroed per call)
    h->fw_mask_off = off; off = align_up(off + (size_t)batch * Hq * n_tiles_cap * n_words * kTileRows * 4);
    h->fw_union_off = off; off = align_up(off + (size_t)batch * Hq * n_tiles_cap * n_words * 4);
    h->fw_fallback_off = off; off = align_up(off + (size_t)batch * Hq * n_tiles_cap * kTileRows * 4);
    h->fw_scratch_off = off; off = align_up(off + (size_t)kExactCtas * kExactWarps * N_ld * 8);
    // digit planes (4 x int8 [B*Hkv*N_ld, 128]) of the mean keys; 128 rows of slack so that the last TMA box
    // stays inside the allocation
    h->fw_kplanes_off = off; off = align_up(off + ((size_t)4 * batch * Hkv * N_ld + 128) * 128);
    // query-gather path: per pair (mode, entries, offset) | per row (entries, first partial) | per row (m, l) of the
    // local range | per key block offsets + work items | entries | partial outputs | partial (m, l)
    {
        const size_t rows_cap = (size_t)batch * Hq * S_cap, n_pairs_cap = ((size_t)S_cap + 255) / 256;
        const uint64_t per_entry = 2ull * D + 16ull + 8ull;      // partial output + (m, l) + entry
        uint64_t cap = h->gather_budget / per_entry;
        // a pair qualifies with at most threshold x (blocks of its union) entries for its 256 rows, and over a causal
        // sequence a pair's union averages half the video's key blocks: threshold x n_cols / 512 entries per row
        double per_row = std::ceil((double)h->gather_pairs_per_block * (double)n_cols / 512.0);
        if (!(per_row < (double)kGatherEntriesPerRow)) per_row = (double)kGatherEntriesPerRow;
        if ((double)cap > (double)rows_cap * per_row) cap = (uint64_t)((double)rows_cap * per_row);
        if (cap > 0xfffffff0ull) cap = 0xfffffff0ull;
        h->gather_cap = (uint32_t)cap;
        h->fw_gpair_off = off; off = align_up(off + (size_t)batch * Hq * n_pairs_cap * 5 * 4);
        h->fw_grow_off = off; off = align_up(off + (cap ? rows_cap * 2 * 4 : 0));
        h->fw_gml_off = off; off = align_up(off + (cap ? rows_cap * 8 : 0));
        h->fw_gitems_off = off; off = align_up(off + (cap ? align_up((n_lists * n_cols * (kGatherClasses + 2) + 2) * 4) + (n_lists * n_cols + cap / 128 + 1) * 16 : 0));
        h->fw_gentries_off = off; off = align_up(off + (size_t)cap * 8);
        h->fw_gparto_off = off; off = align_up(off + (size_t)cap * D * 2);
        h->fw_gpartml_off = off; off = align_up(off + (size_t)cap * 8);
    }
    h->fw_total = off;
    L.forward_workspace_bytes = (int64_t)off;

    // decode workspace: status | bitmaps | block lists | counts | split partials
    // split count: at least ~2 waves of CTAs over the 148 SMs, and among those the count that
    // leaves the last wave fullest (one CTA per SM is resident)
    int splits = 1;
    {
        const long long base = (long long)batch * Hkv;
        double best = -1.0;
        for (int s = 1; s <= 64; ++s) {
            long long ctas = base * s;
            double eff = (double)ctas / (double)((ctas + 147) / 148 * 148);
            if (ctas < 2 * 148 && s < 64) continue;
            if (eff > best + 1e-9) { best = eff; splits = s; }
        }
    }
    h->dc_splits = splits;
    off = 0;
    h->dc_status_off = off; off = align_up(off + 256);
    h->dc_bitmap_off = off; off = align_up(off + (size_t)batch * Hq * n_words * 4);
    h->dc_items_off = off; off = align_up(off + (size_t)batch * Hkv * (S_cap / kBlockTok) * 4);
    h->dc_nitems_off = off; off = align_up(off + (size_t)batch * Hkv * 4);
    h->dc_partial_off = off; off = align_up(off + (size_t)batch * Hkv * splits * (Hq / Hkv) * (D + 2) * 4);
    h->dc_total = off;
    L.decode_workspace_bytes = (int64_t)off;

    h->partitioned = true;
    h->err[0] = 0;
    if (workspace_bytes) *workspace_bytes = h->fw_total > h->dc_total ? h->fw_total : h->dc_total;
    return ADASPARK_OK;
}

adaspark_status_t adaspark_attn_get_layout(const adaspark_attn_t* h, adaspark_attn_layout_t* out_layout) {
    if (!h || !out_layout) return ADASPARK_ERR_INVALID_ARG;
    if (!h->partitioned) return ADASPARK_ERR_NOT_PARTITIONED;
    *out_layout = h->layout;
    return ADASPARK_OK;
}

}  // extern "C"

namespace {

// Prefill of the frames [frame_begin, frame_begin + frame_count) plus, when n_text >= 0 (the last call of a
// sequence), n_text text tokens; n_text < 0: more video follows.  The one-shot forward is the window
// [0, T) with its text.
adaspark_status_t forward_impl(adaspark_attn_t* h, const char* who, const void* q, const void* k, const void* v,
                               int32_t frame_begin, int32_t frame_count, int32_t n_text_arg, int32_t n_prefix, void* out, void* k_cube,
                               void* v_cube, float* cube_keys, uint32_t* sel_bitmap, int32_t* sel_count, void* workspace,
                               size_t workspace_bytes, void* cuda_stream) {
    if (!h) return ADASPARK_ERR_INVALID_ARG;
    if (!h->partitioned) return fail(h, ADASPARK_ERR_NOT_PARTITIONED, "%s: call adaspark_attn_partition first", who);
    if (!k || !v || !k_cube || !v_cube || !cube_keys) return fail(h, ADASPARK_ERR_INVALID_ARG, "%s: NULL k/v/cache pointer", who);
    if ((q == nullptr) != (out == nullptr)) return fail(h, ADASPARK_ERR_INVALID_ARG, "%s: q and out must both be given or both be NULL", who);
    const bool last_call = n_text_arg >= 0;
    const int n_text = last_call ? n_text_arg : 0;
    if (n_prefix < 0 || (long long)n_text + n_prefix > h->n_text_max)
        return fail(h, ADASPARK_ERR_INVALID_ARG, "%s: %d prefix + %d text tokens outside [0, %d]", who, n_prefix, n_text, h->n_text_max);
    const int ct = h->cfg.cube_t;
    const bool whole = frame_begin == 0 && frame_count == h->T;
    if (frame_begin < 0 || frame_count < 0 || frame_begin + frame_count > h->T || frame_begin % ct ||
        ((frame_begin + frame_count) % ct && frame_begin + frame_count != h->T))
        return fail(h, ADASPARK_ERR_INVALID_ARG, "%s: frames [%d, %d) are not whole time blocks of %d frames inside [0, %d)", who,
                    frame_begin, frame_begin + frame_count, ct, h->T);
    if (!whole && (n_prefix > 0 || h->T % ct || h->H % h->cfg.cube_h || h->W % h->cfg.cube_w))
        return fail(h, ADASPARK_ERR_UNSUPPORTED, "%s: a chunked prefill takes no text prefix and needs a grid the cube window divides", who);
    if (last_call && frame_begin + frame_count != h->T)
        return fail(h, ADASPARK_ERR_INVALID_ARG, "%s: the call that brings the text must end the video (frame %d of %d)", who,
                    frame_begin + frame_count, h->T);
    if (frame_count == 0 && n_text == 0) return fail(h, ADASPARK_ERR_INVALID_ARG, "%s: empty call", who);
    if (((long long)frame_begin * h->H * h->W) % 256)
        return fail(h, ADASPARK_ERR_UNSUPPORTED, "%s: a chunk must start at a multiple of 256 tokens (frame_begin * H * W = %lld)", who,
                    (long long)frame_begin * h->H * h->W);
    const bool cache_only = (q == nullptr);
    if (!cache_only) {
        if (!workspace) return fail(h, ADASPARK_ERR_INVALID_ARG, "%s: NULL workspace", who);
        if (workspace_bytes < h->fw_total) return fail(h, ADASPARK_ERR_WORKSPACE_TOO_SMALL, "%s: workspace %zu < %zu bytes", who, workspace_bytes, h->fw_total);
        if ((uintptr_t)workspace % kAlign) return fail(h, ADASPARK_ERR_INVALID_ARG, "%s: workspace not 256-byte aligned", who);
    }
    cudaError_t ce = cudaSetDevice(h->cfg.device);
    if (ce != cudaSuccess) return fail(h, ADASPARK_ERR_CUDA, "%s: cudaSetDevice(%d): %s", who, h->cfg.device, cudaGetErrorString(ce));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    h->launches = 0;
    const Geom g = make_geom(h, n_text, frame_begin, frame_begin + frame_count, n_prefix);
    const int D = g.D;
    auto* kb = (const __nv_bfloat16*)k;
    auto* vb = (const __nv_bfloat16*)v;
    auto* kc = (__nv_bfloat16*)k_cube;
    auto* vc = (__nv_bfloat16*)v_cube;

    // header and head exponents start at zero
    if (!cache_only) cudaMemsetAsync((char*)workspace + h->fw_status_off, 0, h->fw_mask_off - h->fw_status_off, st);
    mark(h, 0, st);
    // K1: re-layout + pooling
    {
        // blocks of this call's rows; the last call of a sequence also zero-fills the cache up to its capacity
        const int blk_begin = g.pos_begin / kBlockTok;
        const int blk_end = last_call ? g.n_kv_blocks_cap : (g.S + kBlockTok - 1) / kBlockTok;
        dim3 grid(blk_end - blk_begin, g.Hkv, g.B);
        uint32_t* slot_valid = (!cache_only && g.ragged) ? (uint32_t*)((char*)workspace + h->fw_valid_off) : nullptr;
        // largest |k|^2 per (batch, kv head): only a call that brings the sequence from its first frame sees every key
        uint32_t* key_norm2 = (!cache_only && frame_begin == 0) ? (uint32_t*)((char*)workspace + h->fw_headmax_off) + g.B * g.Hkv : nullptr;
        if (D == 128) relayout_pool_kernel<128><<<grid, 256, 0, st>>>(g, kb, vb, kc, vc, cube_keys, slot_valid, key_norm2);
        else relayout_pool_kernel<64><<<grid, 256, 0, st>>>(g, kb, vb, kc, vc, cube_keys, slot_valid, key_norm2);
        if (!launch_ok(h, "relayout_pool_kernel")) return ADASPARK_ERR_CUDA;
        const int cube_begin = g.pos_begin >> g.c_shift;
        if (g.C > kBlockTok && g.N_live > cube_begin) {
            pool_large_cubes_kernel<<<dim3(g.N_live - cube_begin, g.Hkv, g.B), D, 0, st>>>(g, kc, cube_keys);
            if (!launch_ok(h, "pool_large_cubes_kernel")) return ADASPARK_ERR_CUDA;
        }
    }
    mark(h, 1, st);
    if (cache_only) return ADASPARK_OK;

    char* ws = (char*)workspace;
    auto* hdr = (adaspark_attn_workspace_header_t*)(ws + h->fw_status_off);
    uint32_t* tile_mask = (uint32_t*)(ws + h->fw_mask_off);
    uint32_t* tile_union = (uint32_t*)(ws + h->fw_union_off);
    auto* qb = (const __nv_bfloat16*)q;

    // K3: scoring + selection
    {
        if (h->sm_count <= 0) {
            int sms = 0;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, h->cfg.device) != cudaSuccess || sms <= 0) sms = 148;
            h->sm_count = sms;
        }
        int32_t* fallback_rows = (int32_t*)(ws + h->fw_fallback_off);
        double* scratch = (double*)(ws + h->fw_scratch_off);
        const bool all = g.top_k <= 0 && !(g.top_p < 1.0);
        auto launch_exact = [&](const int32_t* rows, const uint32_t* n_list, long long n_ids) {
            if (D == 128)
                select_exact_kernel<128><<<kExactCtas, kExactWarps * 32, 0, st>>>(g, qb, cube_keys, rows, n_list, n_ids, scratch,
                                                                                   tile_mask, tile_union, sel_bitmap, sel_count);
            else
                select_exact_kernel<64><<<kExactCtas, kExactWarps * 32, 0, st>>>(g, qb, cube_keys, rows, n_list, n_ids, scratch,
                                                                                  tile_mask, tile_union, sel_bitmap, sel_count);
            return launch_ok(h, "select_exact_kernel");
        };
        if (all) {
            select_all_kernel<<<dim3(g.n_tiles - g.tile_begin, g.Hq, g.B), kTileRows, 0, st>>>(g, tile_mask, tile_union, sel_bitmap, sel_count);
            if (!launch_ok(h, "select_all_kernel")) return ADASPARK_ERR_CUDA;
        }
#ifdef ADASPARK_WITH_TCGEN05
        else if (h->prefill_kernel == 1) {
            uint32_t* head_max = (uint32_t*)(ws + h->fw_headmax_off);
            unsigned char* kplanes = (unsigned char*)(ws + h->fw_kplanes_off);
            const int n_rows = g.B * g.Hkv * g.N_ld;
            key_exponent_kernel<<<dim3(g.B * g.Hkv, 8), 256, 0, st>>>(g, cube_keys, head_max);
            if (!launch_ok(h, "key_exponent_kernel")) return ADASPARK_ERR_CUDA;
            slice_keys_kernel<<<(n_rows + 3) / 4, 128, 0, st>>>(g, cube_keys, head_max, kplanes);
            if (!launch_ok(h, "slice_keys_kernel")) return ADASPARK_ERR_CUDA;
            CUtensorMap tmKs;
            if (!encode_u8_2d(&tmKs, kplanes, (uint64_t)4 * n_rows + 128, kDigitRowBytes, kDigitRowBytes, kScoreTcCols))
                return fail(h, ADASPARK_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed", who);
            const int n_items = g.B * g.Hq * (g.n_tiles - g.tile_begin);
            const int grid = n_items < h->sm_count ? n_items : h->sm_count;
            const bool by_count = g.top_k > 0;
#define ADASPARK_LAUNCH_FUSED(DD, BC)                                                                                  \
    do {                                                                                                               \
        const size_t smem = sizeof(FusedSmem<DD>) + 1024;                                                              \
        if (!set_smem(h, score_select_fused_kernel<DD, BC>, smem, "score_select_fused_kernel")) return ADASPARK_ERR_CUDA; \
        score_select_fused_kernel<DD, BC><<<grid, kFusedThreads, smem, st>>>(                                           \
            g, n_items, qb, tmKs, head_max, tile_mask, tile_union, sel_bitmap, sel_count, fallback_rows,         \
            &hdr->fallback_rows, &hdr->status);                                                                        \
    } while (0)
            if (D == 128) { if (by_count) ADASPARK_LAUNCH_FUSED(128, true); else ADASPARK_LAUNCH_FUSED(128, false); }
            else { if (by_count) ADASPARK_LAUNCH_FUSED(64, true); else ADASPARK_LAUNCH_FUSED(64, false); }
#undef ADASPARK_LAUNCH_FUSED
            if (!launch_ok(h, "score_select_fused_kernel")) return ADASPARK_ERR_CUDA;
            // the rows it left over (normally none): list length is read on the device
            if (!launch_exact(fallback_rows, &hdr->fallback_rows, 0)) return ADASPARK_ERR_CUDA;
        }
#endif
        else {
            cudaMemsetAsync(tile_union, 0, h->fw_fallback_off - h->fw_union_off, st);
            if (!launch_exact(nullptr, nullptr, (long long)g.B * g.Hq * g.n_tiles_cap * kTileRows)) return ADASPARK_ERR_CUDA;
        }
    }

    mark(h, 2, st);
    // K4: gathered attention
#ifdef ADASPARK_WITH_TCGEN05
    if (h->prefill_kernel != 0) {
        // Q tiles are boxes of the caller's tensor [B, S_io, Hq, D] seen as (head x d, x, y, frame, batch) from its first
        // video token on: a box = min(C, 128) cube-major rows = a slab of the cube window
        CUtensorMap tmQ, tmK, tmV;
        uint32_t bx = (uint32_t)(g.cw < 128 ? g.cw : 128), by = (uint32_t)(g.ch < 128 / (int)bx ? g.ch : 128 / (int)bx);
        uint32_t bt = (uint32_t)(g.ct < 128 / (int)(bx * by) ? g.ct : 128 / (int)(bx * by));
        if (bt < 1) bt = 1;
        const uint64_t tok = (uint64_t)g.Hq * D * 2;
        const int frames_here = frame_count > 0 ? frame_count : 1;
        const uint64_t qdims[5] = {(uint64_t)g.Hq * D, (uint64_t)g.W, (uint64_t)g.H, (uint64_t)frames_here, (uint64_t)g.B};
        const uint64_t qstr[4] = {tok, (uint64_t)g.W * tok, (uint64_t)g.H * g.W * tok, (uint64_t)g.S_io * tok};
        const uint32_t qbox[5] = {64u, bx, by, bt, 1u};
        if (!encode_bf16_5d(&tmQ, qb + (size_t)g.n_prefix * g.Hq * D, qdims, qstr, qbox) ||
            !encode_bf16_2d(&tmK, kc, (uint64_t)g.B * g.Hkv * g.S_cap, D, 64, 64) ||
            !encode_bf16_2d(&tmV, vc, (uint64_t)g.B * g.Hkv * g.n_kv_blocks_cap * D, 64, 64, D))
            return fail(h, ADASPARK_ERR_CUDA, "%s: cuTensorMapEncodeTiled failed", who);
        dim3 grid(((g.S + kPairRows - 1) / kPairRows - g.pos_begin / kPairRows) * g.Hq * g.B);
        const uint32_t* slot_valid_c = (const uint32_t*)(ws + h->fw_valid_off);
        // query-gather path for pairs of query tiles with sparse selections (off for p >= 1: nothing is skipped)
        const bool all_sel = g.top_k <= 0 && !(g.top_p < 1.0);
        const bool gather = h->prefill_kernel == 1 && !all_sel && h->gather_cap > 0 && h->gather_pairs_per_block > 0.f;
        GatherWs gw;
        std::memset(&gw, 0, sizeof(gw));
        if (gather) {
            const size_t n_cols = (size_t)(g.S_v + kBlockTok - 1) / kBlockTok;
            const size_t n_lists = (size_t)h->gather_windows * g.B * g.Hkv, n_col_all = n_lists * n_cols;
            const int n_pairs_win = (g.S + kPairRows - 1) / kPairRows - g.pos_begin / kPairRows;
            const size_t rows_cap = (size_t)g.B * g.Hq * g.S_cap, n_pairs_cap = ((size_t)g.S_cap + 255) / 256;
            const size_t n_pair_all = (size_t)g.B * g.Hq * n_pairs_cap;
            gw.ctrl = &hdr->gather_entries;
            gw.pair_mode = (uint32_t*)(ws + h->fw_gpair_off);
            gw.pair_cnt = gw.pair_mode + n_pair_all;
            gw.pair_off = gw.pair_cnt + n_pair_all;
            gw.pair_u = gw.pair_off + n_pair_all;
            gw.pair_list = gw.pair_u + n_pair_all;
            gw.row_cnt = (uint32_t*)(ws + h->fw_grow_off);
            gw.row_ptr = gw.row_cnt + rows_cap;
            gw.col_cnt = (uint32_t*)(ws + h->fw_gcol_off);
            gw.col_cur = gw.col_cnt + n_col_all * kGatherClasses;
            gw.col_roff = (uint32_t*)(ws + h->fw_gitems_off);
            gw.col_off = gw.col_roff + n_col_all * kGatherClasses;
            gw.col_item = gw.col_off + n_col_all + 1;
            gw.items = (uint4*)(ws + h->fw_gitems_off + align_up((n_col_all * (kGatherClasses + 2) + 2) * 4));
            gw.entries = (uint32_t*)(ws + h->fw_gentries_off);
            gw.row_slots = gw.entries + h->gather_cap;
            gw.part_o = (__nv_bfloat16*)(ws + h->fw_gparto_off);
            gw.part_ml = (float2*)(ws + h->fw_gpartml_off);
            gw.ml_local = (float2*)(ws + h->fw_gml_off);
            gw.cap_entries = h->gather_cap;
            gw.n_cols = (int)n_cols;
            gw.n_lists = (int)n_lists;
            gw.n_windows = h->gather_windows;
            gw.pairs_per_window = (n_pairs_win + h->gather_windows - 1) / h->gather_windows;
            gw.n_pairs_cap = (int)n_pairs_cap;
            gw.pairs_per_block = h->gather_pairs_per_block;
            gather_count_kernel<<<grid, 256, 0, st>>>(g, gw, tile_mask, tile_union);
            if (!launch_ok(h, "gather_count_kernel")) return ADASPARK_ERR_CUDA;
            gather_scan_kernel<<<1, 1024, 0, st>>>(g, gw);
            if (!launch_ok(h, "gather_scan_kernel")) return ADASPARK_ERR_CUDA;
            const int icta = (int)((n_col_all + 7) / 8);
            gather_items_kernel<<<icta < 4 * h->sm_count ? icta : 4 * h->sm_count, 256, 0, st>>>(g, gw);
            if (!launch_ok(h, "gather_items_kernel")) return ADASPARK_ERR_CUDA;
        }
        const uint32_t* pair_mode_c = gather ? gw.pair_mode : nullptr;
        const uint32_t* key_norm2_c = frame_begin == 0 ? (const uint32_t*)(ws + h->fw_headmax_off) + g.B * g.Hkv : nullptr;
        mark(h, 5, st);
        if (D == 128) {
            size_t smem = sizeof(TcAttnSmem<128>) + 1024;
            if (!set_smem(h, attn_prefill_tc_kernel<128>, smem, "attn_prefill_tc_kernel")) return ADASPARK_ERR_CUDA;
            attn_prefill_tc_kernel<128><<<grid, kTcThreads, smem, st>>>(g, tmQ, qb, tmK, tmV, tile_mask, tile_union, slot_valid_c, pair_mode_c,
                                                                        gw.n_pairs_cap, gw.ml_local, key_norm2_c, (__nv_bfloat16*)out,
                                                                        (unsigned long long*)&hdr->executed_kv_blocks, &hdr->max_tile_kv_blocks, &hdr->status);
        } else {
            size_t smem = sizeof(TcAttnSmem<64>) + 1024;
            if (!set_smem(h, attn_prefill_tc_kernel<64>, smem, "attn_prefill_tc_kernel")) return ADASPARK_ERR_CUDA;
            attn_prefill_tc_kernel<64><<<grid, kTcThreads, smem, st>>>(g, tmQ, qb, tmK, tmV, tile_mask, tile_union, slot_valid_c, pair_mode_c,
                                                                       gw.n_pairs_cap, gw.ml_local, key_norm2_c, (__nv_bfloat16*)out,
                                                                       (unsigned long long*)&hdr->executed_kv_blocks, &hdr->max_tile_kv_blocks, &hdr->status);
        }
        if (!launch_ok(h, "attn_prefill_tc_kernel")) return ADASPARK_ERR_CUDA;
        mark(h, 6, st);
        if (gather) {
            gather_fill_kernel<<<grid, 256, 0, st>>>(g, gw, tile_mask);
            if (!launch_ok(h, "gather_fill_kernel")) return ADASPARK_ERR_CUDA;
            CUtensorMap tmKg;      // one key block per load: box of 64 d x 64 keys (tmK's) serves as it is
            tmKg = tmK;
            const int ggrid = h->sm_count;                      // persistent: one CTA per SM
            const long long n_rows = (long long)g.B * g.Hq * (g.S - g.pos_begin);    // at most: the rows of all pairs
            if (D == 128) {
                const size_t smem = sizeof(GatherSmem<128>) + 1024;
                if (!set_smem(h, attn_gather_kernel<128>, smem, "attn_gather_kernel")) return ADASPARK_ERR_CUDA;
                attn_gather_kernel<128><<<ggrid, kGatherThreads, smem, st>>>(g, gw, tmKg, tmV, qb, slot_valid_c,
                                                                            (unsigned long long*)&hdr->executed_kv_blocks, &hdr->status);
                if (!launch_ok(h, "attn_gather_kernel")) return ADASPARK_ERR_CUDA;
                const long long ctas = (n_rows + 15) / 16;
                gather_merge_kernel<128><<<(unsigned)(ctas < 8ll * h->sm_count ? ctas : 8ll * h->sm_count), 256, 0, st>>>(g, gw, (__nv_bfloat16*)out);
            } else {
                const size_t smem = sizeof(GatherSmem<64>) + 1024;
                if (!set_smem(h, attn_gather_kernel<64>, smem, "attn_gather_kernel")) return ADASPARK_ERR_CUDA;
                attn_gather_kernel<64><<<ggrid, kGatherThreads, smem, st>>>(g, gw, tmKg, tmV, qb, slot_valid_c,
                                                                           (unsigned long long*)&hdr->executed_kv_blocks, &hdr->status);
                if (!launch_ok(h, "attn_gather_kernel")) return ADASPARK_ERR_CUDA;
                const long long ctas = (n_rows + 31) / 32;
                gather_merge_kernel<64><<<(unsigned)(ctas < 8ll * h->sm_count ? ctas : 8ll * h->sm_count), 256, 0, st>>>(g, gw, (__nv_bfloat16*)out);
            }
            if (!launch_ok(h, "gather_merge_kernel")) return ADASPARK_ERR_CUDA;
        }
    } else
#endif
    {
        dim3 grid(g.n_tiles - g.tile_begin, g.Hq, g.B);
        if (D == 128) {
            size_t smem = sizeof(MmaAttnSmem<128>);
            if (!set_smem(h, attn_prefill_mma_kernel<128>, smem, "attn_prefill_mma_kernel")) return ADASPARK_ERR_CUDA;
            attn_prefill_mma_kernel<128><<<grid, 256, smem, st>>>(g, qb, kc, vc, tile_mask, (__nv_bfloat16*)out, (unsigned long long*)&hdr->executed_kv_blocks);
        } else {
            size_t smem = sizeof(MmaAttnSmem<64>);
            if (!set_smem(h, attn_prefill_mma_kernel<64>, smem, "attn_prefill_mma_kernel")) return ADASPARK_ERR_CUDA;
            attn_prefill_mma_kernel<64><<<grid, 256, smem, st>>>(g, qb, kc, vc, tile_mask, (__nv_bfloat16*)out, (unsigned long long*)&hdr->executed_kv_blocks);
        }
        if (!launch_ok(h, "attn_prefill_mma_kernel")) return ADASPARK_ERR_CUDA;
    }
    mark(h, 3, st);
    mark(h, 4, st);
    return ADASPARK_OK;
}

}  // namespace

extern "C" {

adaspark_status_t adaspark_attn_forward(adaspark_attn_t* h, const void* q, const void* k, const void* v,
                                        int32_t n_text, void* out, void* k_cube, void* v_cube, float* cube_keys,
                                        uint32_t* sel_bitmap, int32_t* sel_count, void* workspace,
                                        size_t workspace_bytes, void* cuda_stream) {
    if (!h) return ADASPARK_ERR_INVALID_ARG;
    if (n_text < 0) return fail(h, ADASPARK_ERR_INVALID_ARG, "forward: n_text %d outside [0, %d]", n_text, h->n_text_max);
    return forward_impl(h, "forward", q, k, v, 0, h->partitioned ? h->T : 0, n_text, 0, out, k_cube, v_cube, cube_keys, sel_bitmap,
                        sel_count, workspace, workspace_bytes, cuda_stream);
}

adaspark_status_t adaspark_attn_forward_host(adaspark_attn_t* h, const void* q_host, const void* k_host, const void* v_host,
                                             int32_t n_text, void* out_host, void* q_dev, void* k_dev, void* v_dev,
                                             void* out_dev, void* k_cube, void* v_cube, float* cube_keys, void* workspace,
                                             size_t workspace_bytes, void* cuda_stream) {
    if (!h) return ADASPARK_ERR_INVALID_ARG;
    if (!h->partitioned) return fail(h, ADASPARK_ERR_NOT_PARTITIONED, "forward_host: call adaspark_attn_partition first");
    if (!k_host || !v_host || !k_dev || !v_dev) return fail(h, ADASPARK_ERR_INVALID_ARG, "forward_host: NULL k/v buffer");
    if ((q_host == nullptr) != (out_host == nullptr) || (q_host != nullptr && (!q_dev || !out_dev)))
        return fail(h, ADASPARK_ERR_INVALID_ARG, "forward_host: q/out host and device buffers must be given together");
    if (n_text < 0 || n_text > h->n_text_max) return fail(h, ADASPARK_ERR_INVALID_ARG, "forward_host: n_text %d outside [0, %d]", n_text, h->n_text_max);
    cudaError_t ce = cudaSetDevice(h->cfg.device);
    if (ce != cudaSuccess) return fail(h, ADASPARK_ERR_CUDA, "forward_host: cudaSetDevice(%d): %s", h->cfg.device, cudaGetErrorString(ce));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t S = (size_t)h->T * h->H * h->W + n_text, D = h->cfg.head_dim;
    const size_t q_bytes = (size_t)h->B * S * h->cfg.n_q_heads * D * 2, kv_bytes = (size_t)h->B * S * h->cfg.n_kv_heads * D * 2;
    if (q_host) ce = cudaMemcpyAsync(q_dev, q_host, q_bytes, cudaMemcpyHostToDevice, st);
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(k_dev, k_host, kv_bytes, cudaMemcpyHostToDevice, st);
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(v_dev, v_host, kv_bytes, cudaMemcpyHostToDevice, st);
    if (ce != cudaSuccess) return fail(h, ADASPARK_ERR_CUDA, "forward_host: host-to-device copy: %s", cudaGetErrorString(ce));
    adaspark_status_t rc = forward_impl(h, "forward_host", q_host ? q_dev : nullptr, k_dev, v_dev, 0, h->T, n_text, 0,
                                        q_host ? out_dev : nullptr, k_cube, v_cube, cube_keys, nullptr, nullptr, workspace,
                                        workspace_bytes, cuda_stream);
    if (rc != ADASPARK_OK) return rc;
    if (q_host) {
        ce = cudaMemcpyAsync(out_host, out_dev, q_bytes, cudaMemcpyDeviceToHost, st);
        if (ce != cudaSuccess) return fail(h, ADASPARK_ERR_CUDA, "forward_host: device-to-host copy: %s", cudaGetErrorString(ce));
    }
    return ADASPARK_OK;
}

adaspark_status_t adaspark_attn_forward_prefix(adaspark_attn_t* h, const void* q, const void* k, const void* v,
                                               int32_t n_prefix, int32_t n_text, void* out, void* k_cube, void* v_cube,
                                               float* cube_keys, uint32_t* sel_bitmap, int32_t* sel_count,
                                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!h) return ADASPARK_ERR_INVALID_ARG;
    if (n_text < 0 || n_prefix < 0) return fail(h, ADASPARK_ERR_INVALID_ARG, "forward_prefix: negative token count");
    return forward_impl(h, "forward_prefix", q, k, v, 0, h->partitioned ? h->T : 0, n_text, n_prefix, out, k_cube, v_cube, cube_keys,
                        sel_bitmap, sel_count, workspace, workspace_bytes, cuda_stream);
}

adaspark_status_t adaspark_attn_forward_chunk(adaspark_attn_t* h, const void* q, const void* k, const void* v,
                                              int32_t frame_begin, int32_t frame_count, int32_t n_text, void* out,
                                              void* k_cube, void* v_cube, float* cube_keys, uint32_t* sel_bitmap,
                                              int32_t* sel_count, void* workspace, size_t workspace_bytes,
                                              void* cuda_stream) {
    return forward_impl(h, "forward_chunk", q, k, v, frame_begin, frame_count, n_text < 0 ? -1 : n_text, 0, out, k_cube, v_cube,
                        cube_keys, sel_bitmap, sel_count, workspace, workspace_bytes, cuda_stream);
}

adaspark_status_t adaspark_attn_decode(adaspark_attn_t* h, const void* q_new, const void* k_new, const void* v_new,
                                       void* k_cube, void* v_cube, const float* cube_keys, const int32_t* text_len,
                                       void* out, uint32_t* sel_bitmap, void* workspace, size_t workspace_bytes,
                                       void* cuda_stream) {
    if (!h) return ADASPARK_ERR_INVALID_ARG;
    if (!h->partitioned) return fail(h, ADASPARK_ERR_NOT_PARTITIONED, "decode: call adaspark_attn_partition first");
    if (!q_new || !k_cube || !v_cube || !cube_keys || !text_len || !out || !workspace)
        return fail(h, ADASPARK_ERR_INVALID_ARG, "decode: NULL pointer");
    if ((k_new == nullptr) != (v_new == nullptr)) return fail(h, ADASPARK_ERR_INVALID_ARG, "decode: k_new and v_new must both be given or both be NULL");
    if (workspace_bytes < h->dc_total) return fail(h, ADASPARK_ERR_WORKSPACE_TOO_SMALL, "decode: workspace %zu < %zu bytes", workspace_bytes, h->dc_total);
    if ((uintptr_t)workspace % kAlign) return fail(h, ADASPARK_ERR_INVALID_ARG, "decode: workspace not 256-byte aligned");
    cudaError_t ce = cudaSetDevice(h->cfg.device);
    if (ce != cudaSuccess) return fail(h, ADASPARK_ERR_CUDA, "decode: cudaSetDevice(%d): %s", h->cfg.device, cudaGetErrorString(ce));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    h->launches = 0;
    const Geom g = make_geom(h, h->n_text_max);
    const int D = g.D;
    char* ws = (char*)workspace;
    auto* hdr = (adaspark_attn_workspace_header_t*)(ws + h->dc_status_off);
    int32_t* status = &hdr->status;
    cudaMemsetAsync(hdr, 0, 256, st);
    mark(h, 0, st);
    uint32_t* dec_bitmap = (uint32_t*)(ws + h->dc_bitmap_off);
    int32_t* items = (int32_t*)(ws + h->dc_items_off);
    int32_t* n_items = (int32_t*)(ws + h->dc_nitems_off);
    float* partial = (float*)(ws + h->dc_partial_off);
    auto* kc = (__nv_bfloat16*)k_cube;
    auto* vc = (__nv_bfloat16*)v_cube;
    auto* qn = (const __nv_bfloat16*)q_new;

    mark(h, 1, st);
    {
        size_t smem = decode_select_smem_bytes(g.N_ld, g.G, g.n_words);
        auto* blocks = (unsigned long long*)&hdr->decode_kv_blocks;
        if (D == 128) {
            if (!set_smem(h, decode_select_plan_kernel<128>, smem, "decode_select_plan_kernel")) return ADASPARK_ERR_CUDA;
            decode_select_plan_kernel<128><<<dim3(g.Hkv, g.B), 256, smem, st>>>(g, qn, (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, kc, vc, cube_keys, text_len, dec_bitmap, sel_bitmap, items, n_items, blocks, status);
        } else {
            if (!set_smem(h, decode_select_plan_kernel<64>, smem, "decode_select_plan_kernel")) return ADASPARK_ERR_CUDA;
            decode_select_plan_kernel<64><<<dim3(g.Hkv, g.B), 256, smem, st>>>(g, qn, (const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, kc, vc, cube_keys, text_len, dec_bitmap, sel_bitmap, items, n_items, blocks, status);
        }
        if (!launch_ok(h, "decode_select_plan_kernel")) return ADASPARK_ERR_CUDA;
    }
    mark(h, 2, st);
    {
        CUtensorMap tmK, tmV;
        if (!encode_bf16_2d(&tmK, kc, (uint64_t)g.B * g.Hkv * g.S_cap, D, 64, 64) ||
            !encode_bf16_2d(&tmV, vc, (uint64_t)g.B * g.Hkv * g.n_kv_blocks_cap * D, 64, 64, D))
            return fail(h, ADASPARK_ERR_CUDA, "decode: cuTensorMapEncodeTiled failed");
        dim3 grid(h->dc_splits, g.Hkv, g.B);
        if (D == 128) {
            size_t smem = sizeof(DecodeSmem<128>) + 1024;
            if (!set_smem(h, decode_splitkv_kernel<128>, smem, "decode_splitkv_kernel")) return ADASPARK_ERR_CUDA;
            decode_splitkv_kernel<128><<<grid, kDecodeThreads, smem, st>>>(g, h->dc_splits, tmK, tmV, qn, dec_bitmap, text_len, items, n_items, partial, status);
        } else {
            size_t smem = sizeof(DecodeSmem<64>) + 1024;
            if (!set_smem(h, decode_splitkv_kernel<64>, smem, "decode_splitkv_kernel")) return ADASPARK_ERR_CUDA;
            decode_splitkv_kernel<64><<<grid, kDecodeThreads, smem, st>>>(g, h->dc_splits, tmK, tmV, qn, dec_bitmap, text_len, items, n_items, partial, status);
        }
        if (!launch_ok(h, "decode_splitkv_kernel")) return ADASPARK_ERR_CUDA;
    }
    mark(h, 3, st);
    decode_combine_kernel<<<dim3(g.Hq, g.B), D, 0, st>>>(g, h->dc_splits, partial, (__nv_bfloat16*)out);
    if (!launch_ok(h, "decode_combine_kernel")) return ADASPARK_ERR_CUDA;
    mark(h, 4, st);
    return ADASPARK_OK;
}

adaspark_status_t adaspark_attn_destroy(adaspark_attn_t* h) {
    if (h && h->timing)
        for (int i = 0; i < 7; ++i) cudaEventDestroy(h->ev[i]);
    delete h;
    return ADASPARK_OK;
}

adaspark_status_t adaspark_attn_enable_stage_timing(adaspark_attn_t* h, int32_t enable) {
    if (!h) return ADASPARK_ERR_INVALID_ARG;
    if (enable && !h->timing) {
        cudaError_t ce = cudaSetDevice(h->cfg.device);
        for (int i = 0; i < 7 && ce == cudaSuccess; ++i) ce = cudaEventCreate(&h->ev[i]);
        if (ce != cudaSuccess) return fail(h, ADASPARK_ERR_CUDA, "enable_stage_timing: %s", cudaGetErrorString(ce));
        h->timing = true;
        h->ev_recorded = false;
    } else if (!enable && h->timing) {
        for (int i = 0; i < 7; ++i) cudaEventDestroy(h->ev[i]);
        h->timing = false;
    }
    return ADASPARK_OK;
}

adaspark_status_t adaspark_attn_get_stage_times(adaspark_attn_t* h, float* ms_out) {
    if (!h || !ms_out) return ADASPARK_ERR_INVALID_ARG;
    if (!h->timing || !h->ev_recorded) return fail(h, ADASPARK_ERR_INVALID_ARG, "get_stage_times: no timed call recorded");
    cudaError_t ce = cudaEventSynchronize(h->ev[4]);
    for (int i = 0; i < 4 && ce == cudaSuccess; ++i) ce = cudaEventElapsedTime(&ms_out[i], h->ev[i], h->ev[i + 1]);
    if (ce != cudaSuccess) return fail(h, ADASPARK_ERR_CUDA, "get_stage_times: %s", cudaGetErrorString(ce));
    return ADASPARK_OK;
}

adaspark_status_t adaspark_attn_get_attention_kernel_ms(adaspark_attn_t* h, float* ms_out) {
    if (!h || !ms_out) return ADASPARK_ERR_INVALID_ARG;
    if (!h->timing || !h->ev_recorded || h->prefill_kernel == 0) return fail(h, ADASPARK_ERR_INVALID_ARG, "get_attention_kernel_ms: no timed tcgen05 prefill recorded");
    cudaError_t ce = cudaEventSynchronize(h->ev[6]);
    if (ce == cudaSuccess) ce = cudaEventElapsedTime(ms_out, h->ev[5], h->ev[6]);
    if (ce != cudaSuccess) return fail(h, ADASPARK_ERR_CUDA, "get_attention_kernel_ms: %s", cudaGetErrorString(ce));
    return ADASPARK_OK;
}

const char* adaspark_attn_last_error(const adaspark_attn_t* h) { return h ? h->err : ""; }

int64_t adaspark_attn_last_launch_count(const adaspark_attn_t* h) { return h ? h->launches : 0; }

adaspark_status_t adaspark_attn_set_prefill_kernel(adaspark_attn_t* h, int32_t which) {
    if (!h) return ADASPARK_ERR_INVALID_ARG;
#ifdef ADASPARK_WITH_TCGEN05
    if (which < 0 || which > 2) return fail(h, ADASPARK_ERR_UNSUPPORTED, "set_prefill_kernel: unknown kernel %d", which);
#else
    if (which != 0) return fail(h, ADASPARK_ERR_UNSUPPORTED, "set_prefill_kernel: kernel %d not built", which);
#endif
    h->prefill_kernel = which;
    return ADASPARK_OK;
}

adaspark_status_t adaspark_attn_set_gather(adaspark_attn_t* h, float pairs_per_block, uint64_t budget_bytes) {
    if (!h) return ADASPARK_ERR_INVALID_ARG;
    if (!(pairs_per_block >= 0.f)) return fail(h, ADASPARK_ERR_INVALID_ARG, "set_gather: threshold %g is not >= 0", (double)pairs_per_block);
    if (h->partitioned && budget_bytes != h->gather_budget)
        return fail(h, ADASPARK_ERR_INVALID_ARG, "set_gather: the byte budget sizes the workspace; set it before adaspark_attn_partition");
    h->gather_pairs_per_block = pairs_per_block;
    h->gather_budget = budget_bytes;
    return ADASPARK_OK;
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------
// Decode for callers that cannot hand over a workspace (see adaspark_attn_decode_static in the
// header).  The scratch lives in this library image: one fixed array per GPU that loads it.
// In host code `g_decode_scratch` is only a stand-in for the symbol, not a device address, so
// the address is looked up once per device with cudaGetSymbolAddress and cached.
// ---------------------------------------------------------------------------------------------
#include <mutex>

static __device__ __align__(256) unsigned char g_decode_scratch[ADASPARK_ATTN_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
void* g_scratch_addr[kMaxDevices] = {nullptr};
}  // namespace

extern "C" adaspark_status_t adaspark_attn_decode_static(adaspark_attn_t* h, const void* q_new, const void* k_new,
                                                         const void* v_new, void* k_cube, void* v_cube,
                                                         const float* cube_keys, const int32_t* text_len, void* out,
                                                         uint32_t* sel_bitmap, void* cuda_stream) {
    if (!h) return ADASPARK_ERR_INVALID_ARG;
    if (!h->partitioned) return fail(h, ADASPARK_ERR_NOT_PARTITIONED, "decode_static: call adaspark_attn_partition first");
    if (h->dc_total > (size_t)ADASPARK_ATTN_STATIC_SCRATCH_BYTES)
        return fail(h, ADASPARK_ERR_WORKSPACE_TOO_SMALL,
                    "decode_static: this partition needs %zu bytes of decode scratch but the built-in scratch holds "
                    "only %zu; use adaspark_attn_decode with a caller workspace",
                    h->dc_total, (size_t)ADASPARK_ATTN_STATIC_SCRATCH_BYTES);
    const int dev = h->cfg.device;
    if (dev < 0 || dev >= kMaxDevices) return fail(h, ADASPARK_ERR_UNSUPPORTED, "decode_static: device ordinal %d", dev);
    cudaError_t ce = cudaSetDevice(dev);
    if (ce != cudaSuccess) return fail(h, ADASPARK_ERR_CUDA, "decode_static: cudaSetDevice(%d): %s", dev, cudaGetErrorString(ce));
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mutex);
        if (!g_scratch_addr[dev]) {   // first call on this device: resolve the symbol's device address
            void* p = nullptr;
            ce = cudaGetSymbolAddress(&p, g_decode_scratch);
            if (ce != cudaSuccess || !p)
                return fail(h, ADASPARK_ERR_CUDA, "decode_static: cudaGetSymbolAddress: %s", cudaGetErrorString(ce));
            g_scratch_addr[dev] = p;
        }
        scratch = g_scratch_addr[dev];
    }
    return adaspark_attn_decode(h, q_new, k_new, v_new, k_cube, v_cube, cube_keys, text_len, out, sel_bitmap, scratch,
                                (size_t)ADASPARK_ATTN_STATIC_SCRATCH_BYTES, cuda_stream);
}

// ---------------------------------------------------------------------------------------------
// Diagnostics (include/adaspark_attn_debug.h)
// ---------------------------------------------------------------------------------------------
#include "../../include/adaspark_attn_debug.h"
#include "umma_selftest.cuh"

extern "C" adaspark_status_t adaspark_attn_debug_imma_selftest(const void* a, const void* b, int32_t* d_out, int32_t* status,
                                                               void* cuda_stream) {
    if (!a || !b || !d_out || !status) return ADASPARK_ERR_INVALID_ARG;
    CUtensorMap tmA, tmB;
    if (!encode_u8_2d(&tmA, a, 128, 128, 128, 128) || !encode_u8_2d(&tmB, b, 128, 128, 128, 128)) return ADASPARK_ERR_CUDA;
    const size_t smem = sizeof(ImmaSelftestSmem) + 1024;
    if (cudaFuncSetAttribute(imma_selftest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return ADASPARK_ERR_CUDA;
    imma_selftest_kernel<<<1, 128, smem, (cudaStream_t)cuda_stream>>>(tmA, tmB, d_out, status);
    return cudaGetLastError() == cudaSuccess ? ADASPARK_OK : ADASPARK_ERR_CUDA;
}

extern "C" adaspark_status_t adaspark_attn_debug_wait_timeout(uint64_t limit_ns, int32_t* status, uint64_t* waited_ns,
                                                              void* cuda_stream) {
    if (!status || !waited_ns || limit_ns < 1000ull || limit_ns > 100000000ull) return ADASPARK_ERR_INVALID_ARG;
    wait_timeout_selftest_kernel<<<1, 64, 0, (cudaStream_t)cuda_stream>>>((unsigned long long)limit_ns, status,
                                                                          (unsigned long long*)waited_ns);
    return cudaGetLastError() == cudaSuccess ? ADASPARK_OK : ADASPARK_ERR_CUDA;
}

extern "C" int32_t adaspark_attn_debug_fastdiv(int32_t n, int32_t d) {
    if (n < 0 || d <= 0) return -1;
    FastDiv f;
    f.init(d);
    return f.div(n);
}

extern "C" adaspark_status_t adaspark_attn_debug_umma_selftest(const void* a, const void* b, const void* c, float* d_out,
                                                               float* e_out, int32_t* status, void* cuda_stream) {
    if (!a || !b || !c || !d_out || !e_out || !status) return ADASPARK_ERR_INVALID_ARG;
    CUtensorMap tmA, tmB, tmC;
    if (!encode_bf16_2d(&tmA, a, 128, 128, 64, 128) || !encode_bf16_2d(&tmB, b, 128, 128, 64, 128) ||
        !encode_bf16_2d(&tmC, c, 128, 128, 64, 128))
        return ADASPARK_ERR_CUDA;
    const size_t smem = sizeof(SelftestSmem) + 1024;
    if (cudaFuncSetAttribute(umma_selftest_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return ADASPARK_ERR_CUDA;
    umma_selftest_kernel<<<1, 128, smem, (cudaStream_t)cuda_stream>>>(tmA, tmB, tmC, d_out, e_out, status);
    return cudaGetLastError() == cudaSuccess ? ADASPARK_OK : ADASPARK_ERR_CUDA;
}
