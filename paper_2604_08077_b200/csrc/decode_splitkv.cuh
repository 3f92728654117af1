// K6: split-KV attention of the decode step over the listed 64-key blocks (Eq. 3, text rule).
//
// HBM-bound: every listed block (K 64xD + V^T Dx64, bf16, 32 KB at D=128) is read once for all
// heads of the GQA group.  One CTA = one split of one (batch, kv head):
//   warp 4      TMA producer: per block two K panels + one V^T tile (128-byte swizzle) into a
//               3-stage shared-memory ring, completion on mbarriers
//   warps 0-3   each owns 16 of the 64 keys of every block: S = Q K^T and O += P V with
//               mma.sync m16n8k16 (the 16 rows are the group's heads, at most 16), its own
//               online softmax state; the four states are merged once at the end.
// The tensor work per byte is tiny, so the legacy tensor path is ample; what matters is keeping
// many 32 KB tiles in flight per SM with almost no issue overhead.
#pragma once
#include "common.cuh"
#include "tc_common.cuh"

namespace adaspark {

constexpr int kDecodeThreads = 160;
// 3 stages of 32 KB (D = 128): two CTAs fit one SM and overlap each other's set-up and merge phases;
// measured 6.85 TB/s against 5.1 TB/s with 4 stages and one CTA per SM.
constexpr int kDecodeStages = 3;

template <int D>
struct DecodeSmem {
    __nv_bfloat16 k[kDecodeStages][D / 64][kBlockTok][64];   // [stage][d panel][key][64 d], swizzled by TMA
    __nv_bfloat16 vt[kDecodeStages][D][kBlockTok];           // [stage][d][key], swizzled by TMA
    uint64_t full[kDecodeStages], empty[kDecodeStages];
    int abort_flag;
};


// grid (n_splits, Hkv, B).  partial[((b*Hkv+gk)*n_splits + split)*G + row] = {m, l, o[D]}
// (base-2 running max, sum, unnormalised output).
template <int D>
__global__ void __launch_bounds__(kDecodeThreads) decode_splitkv_kernel(
    Geom g, int n_splits, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
    const __nv_bfloat16* __restrict__ q_new, const uint32_t* __restrict__ dec_bitmap,
    const int32_t* __restrict__ text_len, const int32_t* __restrict__ items, const int32_t* __restrict__ n_items,
    float* __restrict__ partial, int32_t* __restrict__ status) {
    extern __shared__ unsigned char dec_smem_raw[];
    DecodeSmem<D>& sm = *reinterpret_cast<DecodeSmem<D>*>((reinterpret_cast<uintptr_t>(dec_smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kKSteps = D / 16, kDTiles = D / 8, kPanels = D / 64;
    constexpr int kRowF = D + 2;
    constexpr uint32_t kStageBytes = 2 * kBlockTok * D * 2;

    const int split = blockIdx.x, gk = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n_it = n_items[b * g.Hkv + gk];
    const int per = (n_it + n_splits - 1) / n_splits;
    const int it0 = min(split * per, n_it), it1 = min(it0 + per, n_it);
    const int32_t* my_items = items + (size_t)(b * g.Hkv + gk) * g.n_kv_blocks_cap;

    if (tid == 0) {
        for (int s = 0; s < kDecodeStages; ++s) {
            tc::mbar_init(&sm.full[s], 1);
            tc::mbar_init(&sm.empty[s], 4);
        }
        sm.abort_flag = 0;
        tc::fence_barrier_init();
    }
    __syncthreads();
    volatile int* abort_flag = &sm.abort_flag;

    float mA = -INFINITY, mB = -INFINITY, lA = 0.f, lB = 0.f;
    float o[kDTiles][4];
#pragma unroll
    for (int i = 0; i < kDTiles; ++i) o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f;
    const int rA = lane >> 2, rB = rA + 8;

    if (warp == 4) {
        if (lane == 0) {
            tc::prefetch_tensormap(&tmK);
            tc::prefetch_tensormap(&tmV);
            const int kv_row0 = (b * g.Hkv + gk) * g.S_cap;
            const int v_row0 = (b * g.Hkv + gk) * g.n_kv_blocks_cap * D;
            for (int it = it0; it < it1; ++it) {
                const int i = it - it0, s = i % kDecodeStages, u = i / kDecodeStages;
                if (!tc::mbar_wait(&sm.empty[s], (u & 1) ^ 1, abort_flag)) break;
                const int kb = my_items[it];
                tc::mbar_arrive_expect_tx(&sm.full[s], kStageBytes);
                for (int p = 0; p < kPanels; ++p)
                    tc::tma_load_2d(&sm.k[s][p][0][0], &tmK, p * 64, kv_row0 + kb * kBlockTok, &sm.full[s]);
                tc::tma_load_2d(&sm.vt[s][0][0], &tmV, 0, v_row0 + kb * D, &sm.full[s]);
            }
        }
    } else {
        const int pos_new = g.S_v + text_len[b];
        // Q fragments: rows = heads of the group (zero beyond G)
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

        for (int it = it0; it < it1; ++it) {
            const int i = it - it0, s = i % kDecodeStages, u = i / kDecodeStages;
            if (!tc::mbar_wait(&sm.full[s], u & 1, abort_flag)) break;
            const int kb = my_items[it];
            const int pk0 = kb * kBlockTok + warp * 16;
            const unsigned char* kst = reinterpret_cast<const unsigned char*>(&sm.k[s][0][0][0]);
            const unsigned char* vst = reinterpret_cast<const unsigned char*>(&sm.vt[s][0][0]);

            float sc[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) sc[nt][0] = sc[nt][1] = sc[nt][2] = sc[nt][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < kKSteps; ++ks) {
                // matrices: (keys 0..7, d lo), (keys 0..7, d hi), (keys 8..15, d lo), (keys 8..15, d hi)
                int row = warp * 16 + (lane & 7) + ((lane >> 4) << 3);
                int chunk = ks * 2 + ((lane >> 3) & 1);            // 16-byte chunk along d (0..D/8)
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3, kst + (chunk >> 3) * (kBlockTok * 128) + sw128(row, chunk & 7));
                mma_bf16_16816(sc[0], qf[ks], b0, b1);
                mma_bf16_16816(sc[1], qf[ks], b2, b3);
            }
            uint32_t wordA = 0, wordB = 0;
            if (pk0 < g.S_v) {
                int w = (pk0 >> g.c_shift) >> 5;
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
                    int cb = (pk >> g.c_shift) & 31;
                    bool held = pk < g.S_v && (!g.ragged || pos_to_io(g, pk) >= 0);   // not an empty slot of a boundary cube
                    bool okA = text_ok || (held && ((wordA >> cb) & 1u));
                    bool okB = text_ok || (held && ((wordB >> cb) & 1u));
                    float va = okA ? sc[nt][e] * g.scale_log2 : -INFINITY;
                    float vb = okB ? sc[nt][2 + e] * g.scale_log2 : -INFINITY;
                    sc[nt][e] = va;
                    sc[nt][2 + e] = vb;
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
                float p0 = fast_exp2(sc[nt][0] - refA), p1 = fast_exp2(sc[nt][1] - refA);
                float p2 = fast_exp2(sc[nt][2] - refB), p3 = fast_exp2(sc[nt][3] - refB);
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
                int row = dp * 16 + (lane & 7) + ((lane >> 4) << 3);   // d
                int chunk = warp * 2 + ((lane >> 3) & 1);              // 8-key chunk
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4(b0, b1, b2, b3, vst + sw128(row, chunk));
                mma_bf16_16816(o[dp * 2], pf, b0, b1);
                mma_bf16_16816(o[dp * 2 + 1], pf, b2, b3);
            }
            __syncwarp();
            if (lane == 0) tc::mbar_arrive(&sm.empty[s]);
        }
    }
    __syncthreads();   // every stage consumed (or the waits gave up): the ring can be reused

    // ---- merge the four warps' (m, l, o) through shared memory, then write the CTA partial
    static_assert(sizeof(sm.k) >= 4 * 16 * kRowF * sizeof(float), "merge buffer must fit the K ring");
    float* red = reinterpret_cast<float*>(&sm.k[0][0][0][0]);   // [4 warps][16 rows][kRowF]
    if (warp < 4) {
        lA += __shfl_xor_sync(0xffffffffu, lA, 1);
        lA += __shfl_xor_sync(0xffffffffu, lA, 2);
        lB += __shfl_xor_sync(0xffffffffu, lB, 1);
        lB += __shfl_xor_sync(0xffffffffu, lB, 2);
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
    float* dst = partial + ((size_t)((b * g.Hkv + gk) * n_splits + split) * g.G) * kRowF;
    for (int idx = tid; idx < g.G * kRowF; idx += kDecodeThreads) {
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
                float scl = (mw == -INFINITY) ? 0.f : fast_exp2(mw - m);
                val += red[((size_t)w * 16 + row) * kRowF + c] * scl;
            }
        }
        dst[idx] = val;
    }
    if (tid == 0 && sm.abort_flag) atomicExch(status, 6);
}

}  // namespace adaspark
