// K5 / K7: decode step = one new text token per sequence (text-token rule after Eq. 3).
//
//   decode_select_plan_kernel  per (b, kv head): appends the new token's K / V to the cube-major caches,
//                              then Eq. 1 scores of all heads of the GQA group against
//                              the N cube keys (fp64 tensor op, the cube keys are read once per
//                              group), Eq. 2 per head, then the list of 64-key blocks to visit =
//                              blocks holding a cube selected by any head of the group + text blocks
//   decode_combine_kernel      log-sum-exp merge of the split-KV partials
// The split-KV attention kernel itself is in decode_splitkv.cuh.
#pragma once
#include "common.cuh"
#include "select_radix.cuh"

namespace adaspark {

// Appends the new token's K / V of one (batch, kv head) to the cube-major caches at text slot
// text_len[b] (the V cache holds every 64-position block transposed).  A text_len outside
// [0, n_text_max] writes nothing (the caller reports status 1).  Called by all threads of a CTA.
__device__ __forceinline__ void decode_append(const Geom& g, int b, int gk, const __nv_bfloat16* __restrict__ k_new,
                                              const __nv_bfloat16* __restrict__ v_new, __nv_bfloat16* __restrict__ k_cube,
                                              __nv_bfloat16* __restrict__ v_cube, const int32_t* __restrict__ text_len) {
    const int tl = text_len[b];
    if (tl < 0 || tl > g.n_text) return;             // g.n_text = n_text_max of the partition
    const int pos = g.S_v + tl, blk = pos / kBlockTok, tok = pos % kBlockTok;
    for (int d = threadIdx.x; d < g.D; d += blockDim.x) {
        const size_t src = ((size_t)b * g.Hkv + gk) * g.D + d;
        k_cube[((size_t)(b * g.Hkv + gk) * g.S_cap + pos) * g.D + d] = k_new[src];
        v_cube[(((size_t)(b * g.Hkv + gk) * g.n_kv_blocks_cap + blk) * g.D + d) * kBlockTok + tok] = v_new[src];
    }
}

// Rows (heads) scored per pass: as many as fit next to each other in shared memory, at most 8
// (the M of mma.m8n8k4).
constexpr int kDecodeCandCap = 256;
__host__ __device__ inline int decode_rows_per_pass(int N_ld) {
    int r = (200 * 1024) / (N_ld * 8 + (kSelHistWords + kDecodeCandCap) * 8);
    return r > 8 ? 8 : (r < 1 ? 1 : r);
}
// dynamic smem of decode_select_plan_kernel: rows_per_pass * (N_ld scores + histogram + candidates)
// words of 8 bytes + G * n_words bitmap words of 4 bytes
__host__ __device__ inline size_t decode_select_smem_bytes(int N_ld, int G, int n_words) {
    return (size_t)decode_rows_per_pass(N_ld) * ((size_t)N_ld + kSelHistWords + kDecodeCandCap) * 8 + (size_t)G * n_words * 4;
}

// grid (Hkv, B), 256 threads.  dynamic smem: rows_per_pass * N_ld doubles + G * n_words words.
// items[(b*Hkv+gk) * n_kv_blocks_cap + i] = index of the i-th block to visit.
template <int D>
__global__ void __launch_bounds__(256) decode_select_plan_kernel(
    Geom g, const __nv_bfloat16* __restrict__ q_new, const __nv_bfloat16* __restrict__ k_new,
    const __nv_bfloat16* __restrict__ v_new, __nv_bfloat16* __restrict__ k_cube, __nv_bfloat16* __restrict__ v_cube,
    const float* __restrict__ cube_keys, const int32_t* __restrict__ text_len, uint32_t* __restrict__ dec_bitmap,
    uint32_t* __restrict__ sel_bitmap, int32_t* __restrict__ items, int32_t* __restrict__ n_items,
    unsigned long long* __restrict__ total_blocks, int32_t* __restrict__ status) {
    extern __shared__ double dsp_smem[];
    const int gk = blockIdx.x, b = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // a text_len outside [0, n_text_max] is reported whether or not a token is appended; the
    // sequence then gets an empty block list and a zero output row
    if (threadIdx.x == 0 && (text_len[b] < 0 || text_len[b] > g.n_text)) atomicExch(status, 1);
    if (k_new != nullptr) decode_append(g, b, gk, k_new, v_new, k_cube, v_cube, text_len);   // read by the next kernel
    const int rpp = decode_rows_per_pass(g.N_ld);
    double* logit = dsp_smem;                                              // [rpp][N_ld]
    unsigned long long* sel_scratch = reinterpret_cast<unsigned long long*>(dsp_smem + (size_t)rpp * g.N_ld);   // [rpp][hist + cand]
    uint32_t* bm = reinterpret_cast<uint32_t*>(sel_scratch + (size_t)rpp * (kSelHistWords + kDecodeCandCap));   // [G][n_words]
    const float* kbase = cube_keys + (size_t)(b * g.Hkv + gk) * g.N * D;
    const int rq = lane >> 2, kq = lane & 3;

    for (int h0 = 0; h0 < g.G; h0 += rpp) {
        // ---- scores: logit[r][j] = scale * <q_(h0+r), kbar_j>.  The head-dim index is permuted
        // the same way for both operands so that each lane reads 4 consecutive elements:
        // k-step 4*S + s' uses d = 16*S + 4*kq + s'.
        double a[D / 4];
        {
            const int hr = h0 + rq;
            const bool live = rq < rpp && hr < g.G;
            const __nv_bfloat16* qsrc = q_new + ((size_t)b * g.Hq + gk * g.G + (live ? hr : 0)) * D;
#pragma unroll
            for (int S = 0; S < D / 16; ++S)
#pragma unroll
                for (int s = 0; s < 4; ++s)
                    a[4 * S + s] = live ? (double)__bfloat162float(qsrc[16 * S + 4 * kq + s]) : 0.0;
        }
        // Two groups of 8 cubes per iteration.  The mean keys stream from HBM and nothing else hides their latency
        // (one CTA per SM, eight warps): the loads of the next iteration are issued before the tensor ops of this
        // one, so that two iterations' worth of bytes are in flight per warp.
        auto load_keys = [&](int c0, float4 (&kv)[2][D / 16]) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int cube = c0 + u * 64 + rq;
                const float* ksrc = kbase + (size_t)(cube < g.N ? cube : 0) * D + 4 * kq;
#pragma unroll
                for (int S = 0; S < D / 16; ++S)
                    kv[u][S] = cube < g.N ? *reinterpret_cast<const float4*>(ksrc + 16 * S) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
        };
        auto score_keys = [&](int c0, const float4 (&kv)[2][D / 16]) {
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if (c0 + u * 64 >= g.N_ld) break;
                double acc[2] = {0.0, 0.0};
#pragma unroll
                for (int S = 0; S < D / 16; ++S) {
                    mma_f64_884(acc, a[4 * S + 0], (double)kv[u][S].x);
                    mma_f64_884(acc, a[4 * S + 1], (double)kv[u][S].y);
                    mma_f64_884(acc, a[4 * S + 2], (double)kv[u][S].z);
                    mma_f64_884(acc, a[4 * S + 3], (double)kv[u][S].w);
                }
                if (rq < rpp) {   // C fragment: row = lane/4, columns 2*(lane%4) + {0,1}
                    logit[(size_t)rq * g.N_ld + c0 + u * 64 + 2 * kq] = acc[0] * g.scale_d;
                    logit[(size_t)rq * g.N_ld + c0 + u * 64 + 2 * kq + 1] = acc[1] * g.scale_d;
                }
            }
        };
        {
            float4 kv_a[2][D / 16], kv_b[2][D / 16];
            int c0 = warp * 8;
            if (c0 < g.N_ld) load_keys(c0, kv_a);
            for (; c0 < g.N_ld; c0 += 256) {
                if (c0 + 128 < g.N_ld) load_keys(c0 + 128, kv_b);
                score_keys(c0, kv_a);
                if (c0 + 128 < g.N_ld) {
                    if (c0 + 256 < g.N_ld) load_keys(c0 + 256, kv_a);
                    score_keys(c0 + 128, kv_b);
                }
            }
        }
        __syncthreads();
        // ---- Eq. 2 for one head per warp
        if (warp < rpp && h0 + warp < g.G) {
            const int hr = h0 + warp, h = gk * g.G + hr;
            double* row = logit + (size_t)warp * g.N_ld;
            unsigned long long* keys = reinterpret_cast<unsigned long long*>(row);
            const int n = g.N;
            unsigned long long bd = 0ull;
            const bool all = g.top_k <= 0 && !(g.top_p < 1.0);
            if (!all) {
                unsigned long long* hist = sel_scratch + (size_t)warp * (kSelHistWords + kDecodeCandCap);
                bd = nucleus_boundary_radix<32, true>(row, n, g.top_p, g.top_k, keys, hist, hist + kSelHistWords, kDecodeCandCap, lane);
            }
            for (int w = 0; w < g.n_words; ++w) {
                int j = w * 32 + lane;
                bool on = j < n && (all || keys[j] >= bd);
                uint32_t word = __ballot_sync(0xffffffffu, on);
                if (lane == 0) {
                    bm[hr * g.n_words + w] = word;
                    dec_bitmap[((size_t)b * g.Hq + h) * g.n_words + w] = word;
                    if (sel_bitmap) sel_bitmap[((size_t)b * g.Hq + h) * g.n_words + w] = word;
                }
            }
        }
        __syncthreads();
    }

    // ---- plan: blocks that hold a selected cube of any head of the group, plus the text blocks
    // (first the union of the group's bitmaps, written over the first head's row)
    for (int w = threadIdx.x; w < g.n_words; w += blockDim.x) {
        uint32_t u = 0;
        for (int i = 0; i < g.G; ++i) u |= bm[i * g.n_words + w];
        bm[w] = u;
    }
    __syncthreads();
    // every warp takes a contiguous run of blocks: count, prefix over the warps, then write
    __shared__ int plan_cnt[8];
    const int tl = text_len[b];
    const int last_pos = g.S_v + tl;                     // position of the new token
    int n_blk = 0;
    if (tl >= 0 && tl <= g.n_text) n_blk = last_pos / kBlockTok + 1;
    const int per_warp = ((n_blk + 7) / 8 + 31) / 32 * 32;
    const int kb_lo = warp * per_warp, kb_hi = min(kb_lo + per_warp, n_blk);
    auto block_needed = [&](int kb) -> bool {
        if (kb >= kb_hi) return false;
        bool need = kb * kBlockTok + kBlockTok - 1 >= g.S_v;   // holds text positions
        if (kb * kBlockTok < g.S_v) {
            int c_lo = (kb * kBlockTok) >> g.c_shift;
            int c_hi = min((kb * kBlockTok + kBlockTok - 1) >> g.c_shift, g.N - 1);
            uint32_t span = c_hi - c_lo + 1;
            uint32_t bits = (span >= 32 ? 0xffffffffu : ((1u << span) - 1u)) << (c_lo & 31);
            if (bm[c_lo >> 5] & bits) need = true;
        }
        return need;
    };
    int mine = 0;
    for (int kb0 = kb_lo; kb0 < kb_hi; kb0 += 32) mine += __popc(__ballot_sync(0xffffffffu, block_needed(kb0 + lane)));
    if (lane == 0) plan_cnt[warp] = mine;
    __syncthreads();
    int count = 0, total = 0;
    for (int i = 0; i < 8; ++i) {
        if (i < warp) count += plan_cnt[i];
        total += plan_cnt[i];
    }
    int32_t* dst = items + (size_t)(b * g.Hkv + gk) * g.n_kv_blocks_cap;
    for (int kb0 = kb_lo; kb0 < kb_hi; kb0 += 32) {
        const int kb = kb0 + lane;
        const bool need = block_needed(kb);
        const uint32_t ball = __ballot_sync(0xffffffffu, need);
        if (need) dst[count + __popc(ball & ((1u << lane) - 1u))] = kb;
        count += __popc(ball);
    }
    if (threadIdx.x == 0) {
        n_items[b * g.Hkv + gk] = total;
        atomicAdd(total_blocks, (unsigned long long)total);
    }
}

// grid (Hq, B), D threads.  partial[((b*Hkv+gk)*n_splits + split)*G + row] = {m, l, o[D]}.
__global__ void decode_combine_kernel(Geom g, int n_splits, const float* __restrict__ partial,
                                      __nv_bfloat16* __restrict__ out) {
    const int h = blockIdx.x, b = blockIdx.y, d = threadIdx.x;
    if (d >= g.D) return;
    const int gk = h / g.G, row = h - gk * g.G;
    const int rowF = g.D + 2;
    const float* base = partial + ((size_t)(b * g.Hkv + gk) * n_splits * g.G + row) * rowF;
    float m = -INFINITY;
    for (int s = 0; s < n_splits; ++s) m = fmaxf(m, base[(size_t)s * g.G * rowF]);
    float l = 0.f, acc = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        const float* p = base + (size_t)s * g.G * rowF;
        float sc = (p[0] == -INFINITY) ? 0.f : exp2f(p[0] - m);
        l += p[1] * sc;
        acc += p[2 + d] * sc;
    }
    out[((size_t)b * g.Hq + h) * g.D + d] = __float2bfloat16(l > 0.f ? acc / l : 0.f);
}

}  // namespace adaspark
