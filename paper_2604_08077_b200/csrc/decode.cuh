// K5-K7: decode step = one new text token per sequence (text-token rule after Eq. 3).
//
//   decode_append_kernel        append the new token's K / V to the cube-major caches
//   decode_score_select_kernel  Eq. 1-2 for the (b, query head) rows against all N cube keys
//   decode_plan_kernel          per (b, kv head): list of 64-token blocks to visit = blocks that
//                               hold a cube selected by any head of the GQA group + text blocks
//   decode_splitkv_kernel       split-KV attention over the listed blocks, per-head masks
//   decode_combine_kernel       log-sum-exp merge of the split partials
// The split-KV kernel is HBM-bound: each listed block (K 64xD + V^T Dx64, bf16) is read once
// for all heads of the group.
#pragma once
#include "common.cuh"
#include "score_select.cuh"
#include "attn_prefill_mma.cuh"   // swz()

namespace adaspark {

constexpr int kDecodeThreads = 128;
constexpr int kDecodeStages = 3;

__global__ void decode_append_kernel(Geom g, const __nv_bfloat16* __restrict__ k_new,
                                     const __nv_bfloat16* __restrict__ v_new,
                                     __nv_bfloat16* __restrict__ k_cube, __nv_bfloat16* __restrict__ v_cube,
                                     const int32_t* __restrict__ text_len, int32_t* __restrict__ status) {
    const int b = blockIdx.x;
    const int tl = text_len[b];
    if (tl < 0 || g.S_v + tl + 1 > g.S_cap) {
        if (threadIdx.x == 0) atomicExch(status, 1);
        return;
    }
    const int pos = g.S_v + tl, blk = pos / kBlockTok, tok = pos % kBlockTok;
    for (int idx = threadIdx.x; idx < g.Hkv * g.D; idx += blockDim.x) {
        int gk = idx / g.D, d = idx - gk * g.D;
        size_t src = ((size_t)b * g.Hkv + gk) * g.D + d;
        k_cube[((size_t)(b * g.Hkv + gk) * g.S_cap + pos) * g.D + d] = k_new[src];
        v_cube[(((size_t)(b * g.Hkv + gk) * g.n_kv_blocks_cap + blk) * g.D + d) * kBlockTok + tok] = v_new[src];
    }
}

// grid (Hq, B), 256 threads.  dynamic smem: N_ld doubles.
__global__ void __launch_bounds__(256) decode_score_select_kernel(Geom g, const __nv_bfloat16* __restrict__ q_new,
                                                                  const float* __restrict__ cube_keys,
                                                                  uint32_t* __restrict__ dec_bitmap,
                                                                  uint32_t* __restrict__ sel_bitmap) {
    extern __shared__ double dsel_smem[];
    const int h = blockIdx.x, b = blockIdx.y, gk = h / g.G;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int per_lane = g.D / 32;                       // 2 or 4
    double qd[4];
    const __nv_bfloat16* qsrc = q_new + ((size_t)b * g.Hq + h) * g.D + lane * per_lane;
    for (int i = 0; i < per_lane; ++i) qd[i] = (double)__bfloat162float(qsrc[i]);
    const float* kb = cube_keys + (size_t)(b * g.Hkv + gk) * g.N * g.D + lane * per_lane;
    for (int j = warp; j < g.N; j += 8) {
        const float* kr = kb + (size_t)j * g.D;
        double acc = 0.0;
        for (int i = 0; i < per_lane; ++i) acc += qd[i] * (double)kr[i];
        acc = warp_sum(acc);
        if (lane == 0) dsel_smem[j] = acc * g.scale_d;
    }
    __syncthreads();
    if (warp != 0) return;
    unsigned long long* keys = reinterpret_cast<unsigned long long*>(dsel_smem);
    const int n = g.N;
    unsigned long long bd = 0ull;
    if (g.top_p < 1.0) {
        double mx = -INFINITY;
        for (int j = lane; j < n; j += 32) mx = fmax(mx, dsel_smem[j]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmax(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        double z = 0.0;
        for (int j = lane; j < n; j += 32) {
            double ej = exp(dsel_smem[j] - mx);
            keys[j] = order_key(ej, j);
            z += ej;
        }
        z = warp_sum(z);
        __syncwarp();
        bd = nucleus_boundary(keys, n, g.top_p * z, lane);
    } else {
        for (int j = lane; j < n; j += 32) keys[j] = order_key(1.0, j);
        __syncwarp();
    }
    for (int w = 0; w < g.n_words; ++w) {
        int j = w * 32 + lane;
        bool on = j < n && keys[j] >= bd;
        uint32_t word = __ballot_sync(0xffffffffu, on);
        if (lane == 0) {
            dec_bitmap[((size_t)b * g.Hq + h) * g.n_words + w] = word;
            if (sel_bitmap) sel_bitmap[((size_t)b * g.Hq + h) * g.n_words + w] = word;
        }
    }
}

// grid (Hkv, B), 32 threads.  items[(b*Hkv+gk) * n_kv_blocks_cap + i] = block index.
__global__ void decode_plan_kernel(Geom g, const uint32_t* __restrict__ dec_bitmap,
                                   const int32_t* __restrict__ text_len, int32_t* __restrict__ items,
                                   int32_t* __restrict__ n_items, unsigned long long* __restrict__ total_blocks) {
    const int gk = blockIdx.x, b = blockIdx.y, lane = threadIdx.x;
    const int tl = text_len[b];
    const int last_pos = g.S_v + tl;                     // position of the new token
    int n_blk = 0;
    if (tl >= 0 && last_pos < g.S_cap) n_blk = last_pos / kBlockTok + 1;
    int32_t* dst = items + (size_t)(b * g.Hkv + gk) * g.n_kv_blocks_cap;
    const uint32_t* bm = dec_bitmap + (size_t)(b * g.Hq + gk * g.G) * g.n_words;
    int count = 0;
    for (int kb0 = 0; kb0 < n_blk; kb0 += 32) {
        int kb = kb0 + lane;
        bool need = false;
        if (kb < n_blk) {
            if (kb * kBlockTok + kBlockTok - 1 >= g.S_v) need = true;   // holds text positions
            if (kb * kBlockTok < g.S_v) {
                int c_lo = (kb * kBlockTok) / g.C;
                int c_hi = min((kb * kBlockTok + kBlockTok - 1) / g.C, g.N - 1);
                uint32_t span = c_hi - c_lo + 1;
                uint32_t bits = (span >= 32 ? 0xffffffffu : ((1u << span) - 1u)) << (c_lo & 31);
                uint32_t u = 0;
                for (int i = 0; i < g.G; ++i) u |= bm[(size_t)i * g.n_words + (c_lo >> 5)];
                if (u & bits) need = true;
            }
        }
        uint32_t ball = __ballot_sync(0xffffffffu, need);
        if (need) dst[count + __popc(ball & ((1u << lane) - 1u))] = kb;
        count += __popc(ball);
    }
    if (lane == 0) {
        n_items[b * g.Hkv + gk] = count;
        atomicAdd(total_blocks, (unsigned long long)count);
    }
}

template <int D>
struct DecodeSmem {
    __nv_bfloat16 k[kDecodeStages][kBlockTok][D];
    __nv_bfloat16 vt[kDecodeStages][D][kBlockTok];
};

// grid (n_splits, Hkv, B), 128 threads; warp w owns tokens 16w..16w+15 of every block.
// partial[((b*Hkv+gk)*n_splits + split)*16 + row] = {m, l, o[D]} (base-2 running max, sum, unnormalised).
template <int D>
__global__ void __launch_bounds__(kDecodeThreads) decode_splitkv_kernel(
    Geom g, int n_splits, const __nv_bfloat16* __restrict__ q_new, const __nv_bfloat16* __restrict__ k_cube,
    const __nv_bfloat16* __restrict__ v_cube, const uint32_t* __restrict__ dec_bitmap,
    const int32_t* __restrict__ text_len, const int32_t* __restrict__ items,
    const int32_t* __restrict__ n_items, float* __restrict__ partial) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    DecodeSmem<D>& sm = *reinterpret_cast<DecodeSmem<D>*>(smem_raw);
    constexpr int kQChunks = D / 8, kKSteps = D / 16, kDTiles = D / 8;
    constexpr int kRowF = D + 2;   // floats per partial row

    const int split = blockIdx.x, gk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_it = n_items[b * g.Hkv + gk];
    const int per = (n_it + n_splits - 1) / n_splits;
    const int it0 = min(split * per, n_it), it1 = min(it0 + per, n_it);
    const int32_t* my_items = items + (size_t)(b * g.Hkv + gk) * g.n_kv_blocks_cap;
    const int pos_new = g.S_v + text_len[b];

    // Q fragments: rows = heads of the group (zero beyond G)
    const int rA = lane >> 2, rB = rA + 8;
    uint32_t qf[kKSteps][4];
    {
        const __nv_bfloat16* qb = q_new + ((size_t)b * g.Hq + gk * g.G) * D;
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
            int c = ks * 16 + 2 * (lane & 3);
            qf[ks][0] = rA < g.G ? *reinterpret_cast<const uint32_t*>(qb + (size_t)rA * D + c) : 0u;
            qf[ks][1] = rB < g.G ? *reinterpret_cast<const uint32_t*>(qb + (size_t)rB * D + c) : 0u;
            qf[ks][2] = rA < g.G ? *reinterpret_cast<const uint32_t*>(qb + (size_t)rA * D + c + 8) : 0u;
            qf[ks][3] = rB < g.G ? *reinterpret_cast<const uint32_t*>(qb + (size_t)rB * D + c + 8) : 0u;
        }
    }
    const uint32_t* bmA = dec_bitmap + (size_t)(b * g.Hq + gk * g.G + (rA < g.G ? rA : 0)) * g.n_words;
    const uint32_t* bmB = dec_bitmap + (size_t)(b * g.Hq + gk * g.G + (rB < g.G ? rB : 0)) * g.n_words;

    const __nv_bfloat16* kbase = k_cube + (size_t)(b * g.Hkv + gk) * g.S_cap * D;
    const __nv_bfloat16* vbase = v_cube + (size_t)(b * g.Hkv + gk) * g.n_kv_blocks_cap * D * kBlockTok;
    auto load_block = [&](int kb, int stage) {
        const __nv_bfloat16* ksrc = kbase + (size_t)kb * kBlockTok * D;
        for (int idx = tid; idx < kBlockTok * kQChunks; idx += kDecodeThreads) {
            int row = idx / kQChunks, c = idx - row * kQChunks;
            cp_async_16(&sm.k[stage][row][swz(row, c) * 8], ksrc + (size_t)row * D + c * 8);
        }
        const __nv_bfloat16* vsrc = vbase + (size_t)kb * D * kBlockTok;
        for (int idx = tid; idx < D * 8; idx += kDecodeThreads) {
            int row = idx >> 3, c = idx & 7;
            cp_async_16(&sm.vt[stage][row][swz(row, c) * 8], vsrc + (size_t)row * kBlockTok + c * 8);
        }
    };

    float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
    float o[kDTiles][4];
#pragma unroll
    for (int i = 0; i < kDTiles; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;

    // prologue: fill stages-1 slots
#pragma unroll
    for (int s = 0; s < kDecodeStages - 1; ++s) {
        if (it0 + s < it1) load_block(my_items[it0 + s], s);
        cp_async_commit();
    }
    for (int it = it0; it < it1; ++it) {
        const int stage = (it - it0) % kDecodeStages;
        {
            int nxt = it + kDecodeStages - 1;
            if (nxt < it1) load_block(my_items[nxt], (nxt - it0) % kDecodeStages);
            cp_async_commit();
        }
        cp_async_wait<kDecodeStages - 1>();
        __syncthreads();
        const int kb = my_items[it];
        const int pk0 = kb * kBlockTok + warp * 16;

        float s[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < kKSteps; ++ks) {
            int row = warp * 16 + (lane & 7) + ((lane >> 4) << 3);
            int chunk = ks * 2 + ((lane >> 3) & 1);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(b0, b1, b2, b3, &sm.k[stage][row][swz(row, chunk) * 8]);
            mma_bf16_16816(s[0], qf[ks], b0, b1);
            mma_bf16_16816(s[1], qf[ks], b2, b3);
        }
        uint32_t wordA = 0, wordB = 0;
        if (pk0 < g.S_v) {
            int w = (pk0 / g.C) >> 5;
            wordA = bmA[w];
            wordB = bmB[w];
        }
        float mxA = -INFINITY, mxB = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                int pk = pk0 + nt * 8 + 2 * (lane & 3) + e;
                bool text_ok = pk >= g.S_v && pk <= pos_new;
                bool okA = text_ok || (pk < g.S_v && ((wordA >> ((pk / g.C) & 31)) & 1u));
                bool okB = text_ok || (pk < g.S_v && ((wordB >> ((pk / g.C) & 31)) & 1u));
                float va = okA ? s[nt][e] * g.scale_log2 : -INFINITY;
                float vb = okB ? s[nt][2 + e] * g.scale_log2 : -INFINITY;
                s[nt][e] = va;
                s[nt][2 + e] = vb;
                mxA = fmaxf(mxA, va);
                mxB = fmaxf(mxB, vb);
            }
        mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 1));
        mxA = fmaxf(mxA, __shfl_xor_sync(0xffffffffu, mxA, 2));
        mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 1));
        mxB = fmaxf(mxB, __shfl_xor_sync(0xffffffffu, mxB, 2));
        float mA_new = fmaxf(mA, mxA), mB_new = fmaxf(mB, mxB);
        float refA = (mA_new == -INFINITY) ? 0.f : mA_new;
        float refB = (mB_new == -INFINITY) ? 0.f : mB_new;
        float corrA = fast_exp2(mA - refA), corrB = fast_exp2(mB - refB);
        mA = mA_new;
        mB = mB_new;
        uint32_t pf[4];
        float sumA = 0.f, sumB = 0.f;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
            float p0 = fast_exp2(s[nt][0] - refA), p1 = fast_exp2(s[nt][1] - refA);
            float p2 = fast_exp2(s[nt][2] - refB), p3 = fast_exp2(s[nt][3] - refB);
            sumA += p0 + p1;
            sumB += p2 + p3;
            pf[nt * 2 + 0] = pack_bf16x2(p0, p1);
            pf[nt * 2 + 1] = pack_bf16x2(p2, p3);
        }
        lA = lA * corrA + sumA;
        lB = lB * corrB + sumB;
#pragma unroll
        for (int dt = 0; dt < kDTiles; ++dt) {
            o[dt][0] *= corrA; o[dt][1] *= corrA;
            o[dt][2] *= corrB; o[dt][3] *= corrB;
        }
#pragma unroll
        for (int dp = 0; dp < kDTiles / 2; ++dp) {
            int row = dp * 16 + (lane & 7) + ((lane >> 4) << 3);
            int chunk = warp * 2 + ((lane >> 3) & 1);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(b0, b1, b2, b3, &sm.vt[stage][row][swz(row, chunk) * 8]);
            mma_bf16_16816(o[dp * 2], pf, b0, b1);
            mma_bf16_16816(o[dp * 2 + 1], pf, b2, b3);
        }
        __syncthreads();
    }
    cp_async_wait<0>();
    __syncthreads();

    // ---- merge the four warps' (m, l, o) through shared memory, then write the CTA partial
    lA += __shfl_xor_sync(0xffffffffu, lA, 1);
    lA += __shfl_xor_sync(0xffffffffu, lA, 2);
    lB += __shfl_xor_sync(0xffffffffu, lB, 1);
    lB += __shfl_xor_sync(0xffffffffu, lB, 2);
    float* red = reinterpret_cast<float*>(smem_raw);   // [4 warps][16 rows][kRowF]
    {
        float* ra = red + ((size_t)warp * 16 + rA) * kRowF;
        float* rb = red + ((size_t)warp * 16 + rB) * kRowF;
        if ((lane & 3) == 0) { ra[0] = mA; ra[1] = lA; rb[0] = mB; rb[1] = lB; }
#pragma unroll
        for (int dt = 0; dt < kDTiles; ++dt) {
            int d = dt * 8 + 2 * (lane & 3);
            ra[2 + d] = o[dt][0]; ra[2 + d + 1] = o[dt][1];
            rb[2 + d] = o[dt][2]; rb[2 + d + 1] = o[dt][3];
        }
    }
    __syncthreads();
    float* dst = partial + ((size_t)((b * g.Hkv + gk) * n_splits + split) * 16) * kRowF;
    for (int idx = tid; idx < 16 * kRowF; idx += kDecodeThreads) {
        int row = idx / kRowF, c = idx - row * kRowF;
        float m = -INFINITY;
        for (int w = 0; w < 4; ++w) m = fmaxf(m, red[((size_t)w * 16 + row) * kRowF]);
        float val;
        if (c == 0) {
            val = m;
        } else {
            val = 0.f;
            for (int w = 0; w < 4; ++w) {
                float mw = red[((size_t)w * 16 + row) * kRowF];
                float sc = (mw == -INFINITY) ? 0.f : fast_exp2(mw - m);
                val += red[((size_t)w * 16 + row) * kRowF + c] * sc;
            }
        }
        dst[idx] = val;
    }
}

// grid (Hq, B), D threads.
__global__ void decode_combine_kernel(Geom g, int n_splits, const float* __restrict__ partial,
                                      __nv_bfloat16* __restrict__ out) {
    const int h = blockIdx.x, b = blockIdx.y, d = threadIdx.x;
    if (d >= g.D) return;
    const int gk = h / g.G, row = h - gk * g.G;
    const int rowF = g.D + 2;
    const float* base = partial + ((size_t)(b * g.Hkv + gk) * n_splits * 16 + row) * rowF;
    float m = -INFINITY;
    for (int s = 0; s < n_splits; ++s) m = fmaxf(m, base[(size_t)s * 16 * rowF]);
    float l = 0.f, acc = 0.f;
    for (int s = 0; s < n_splits; ++s) {
        const float* p = base + (size_t)s * 16 * rowF;
        float sc = (p[0] == -INFINITY) ? 0.f : exp2f(p[0] - m);
        l += p[1] * sc;
        acc += p[2 + d] * sc;
    }
    out[((size_t)b * g.Hq + h) * g.D + d] = __float2bfloat16(l > 0.f ? acc / l : 0.f);
}

}  // namespace adaspark
