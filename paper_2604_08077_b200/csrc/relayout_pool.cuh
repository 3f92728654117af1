// K1: cube-major re-layout of K and V (Algorithm 1, "Reshape K,V into Cubes") fused with the
// per-cube mean key (Sec. 3.2, definition under Eq. 1).  HBM-bound: every K/V element is read
// once and written once.
//
// One CTA handles one block of 64 consecutive cube-major positions of one (batch, kv head):
//   k_cube [B,Hkv,S_cap,D]        row pos            <- K[b, raster(pos), g, :]
//   v_cube [B,Hkv,S_cap/64,D,64]  block blk, V^T     <- V[b, raster(blk*64 + tok), g, d]
//   cube_keys [B,Hkv,N,D] fp32    mean over the C keys of each cube inside the block (C <= 64);
//                                 cubes larger than a block are pooled by pool_large_cubes_kernel.
// Positions >= S are zero-filled so that later tensor-core reads never meet non-finite data.
// The kernel also leaves the largest |k|^2 of every (batch, kv head) among the rows it wrote (float bits,
// atomic maximum): with |q| it bounds every score of a query row (Cauchy-Schwarz), which lets the attention
// kernel fix a row's softmax reference in advance.
#pragma once
#include "common.cuh"

namespace adaspark {

// Tokens a cube holds: C, fewer at the far faces of a grid the window does not divide.
__device__ __forceinline__ int cube_tokens_held(const Geom& g, int cube) {
    if (!g.ragged) return g.C;
    int cx, cy, cb, t;
    g.div_nW.divmod(cube, t, cx);
    g.div_nH.divmod(t, cb, cy);
    return min(g.ct, g.T - cb * g.ct) * min(g.ch, g.H - cy * g.ch) * min(g.cw, g.W - cx * g.cw);
}

template <int D>
__global__ void __launch_bounds__(256) relayout_pool_kernel(Geom g, const __nv_bfloat16* __restrict__ k,
                                                            const __nv_bfloat16* __restrict__ v,
                                                            __nv_bfloat16* __restrict__ k_cube,
                                                            __nv_bfloat16* __restrict__ v_cube,
                                                            float* __restrict__ cube_keys,
                                                            uint32_t* __restrict__ slot_valid,
                                                            uint32_t* __restrict__ key_norm2_bits) {
    constexpr int kChunks = D / 8;    // 16-byte chunks per row
    constexpr int kVPitch = D + 2;    // padded pitch (elements) of the V staging tile
    __shared__ __align__(16) __nv_bfloat16 Ks[kBlockTok][D];
    __shared__ __align__(16) __nv_bfloat16 Vs[kBlockTok][kVPitch];

    const int blk = blockIdx.x + g.pos_begin / kBlockTok, gk = blockIdx.y, b = blockIdx.z;   // blocks of this call's row window
    const int pos0 = blk * kBlockTok;
    const int tid = threadIdx.x;
    float row_max = 0.f;

    for (int idx = tid; idx < kBlockTok * kChunks; idx += 256) {
        int row = idx / kChunks, c = idx - row * kChunks;
        int pos = pos0 + row;
        uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
        if (slot_live(g, pos)) {
            size_t src = (io_row(g, b, pos) * g.Hkv + gk) * D + c * 8;
            kv4 = *reinterpret_cast<const uint4*>(k + src);
            vv4 = *reinterpret_cast<const uint4*>(v + src);
        }
        *reinterpret_cast<uint4*>(&Ks[row][c * 8]) = kv4;
        *reinterpret_cast<uint4*>(k_cube + ((size_t)(b * g.Hkv + gk) * g.S_cap + pos) * D + c * 8) = kv4;
        if (key_norm2_bits != nullptr) {
            // |k|^2 of the row: the kChunks consecutive lanes that hold it add their parts (64 * kChunks is a
            // multiple of 256, so every lane of the warp is here); non-negative floats order like their bits
            const uint32_t w[4] = {kv4.x, kv4.y, kv4.z, kv4.w};
            float n2 = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float lo = __uint_as_float(w[i] << 16), hi = __uint_as_float(w[i] & 0xffff0000u);
                n2 = fmaf(lo, lo, fmaf(hi, hi, n2));
            }
#pragma unroll
            for (int o = kChunks / 2; o > 0; o >>= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
            row_max = fmaxf(row_max, n2);
        }
        uint32_t* vdst = reinterpret_cast<uint32_t*>(&Vs[row][c * 8]);
        vdst[0] = vv4.x; vdst[1] = vv4.y; vdst[2] = vv4.z; vdst[3] = vv4.w;
    }
    if (key_norm2_bits != nullptr) {
        const uint32_t m = __reduce_max_sync(0xffffffffu, __float_as_uint(row_max));
        if ((tid & 31) == 0 && m) atomicMax(key_norm2_bits + b * g.Hkv + gk, m);
    }
    __syncthreads();

    // Which of the block's 64 slots hold a token (two words per block; read by the attention kernels of a
    // ragged grid, whose boundary cubes have empty slots)
    if (slot_valid != nullptr && gk == 0 && b == 0 && tid < 64) {
        const uint32_t bits = __ballot_sync(0xffffffffu, slot_live(g, pos0 + tid));
        if ((tid & 31) == 0) slot_valid[2 * blk + (tid >> 5)] = bits;
    }

    // V^T: 8 consecutive threads write one 128-byte row (64 tokens of one d).
    __nv_bfloat16* vt = v_cube + ((size_t)(b * g.Hkv + gk) * g.n_kv_blocks_cap + blk) * D * kBlockTok;
    for (int idx = tid; idx < D * 8; idx += 256) {
        int d = idx >> 3, tc = idx & 7;
        __align__(16) __nv_bfloat16 tmp[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) tmp[i] = Vs[tc * 8 + i][d];
        *reinterpret_cast<uint4*>(vt + d * kBlockTok + tc * 8) = *reinterpret_cast<uint4*>(tmp);
    }

    // Mean keys of the cubes that lie inside this block (exact fp64 sum, one rounding to fp32).
    if (g.C <= kBlockTok && pos0 < g.S_v) {
        int cubes_here = kBlockTok / g.C;
        for (int idx = tid; idx < cubes_here * D; idx += 256) {
            int cb = idx / D, d = idx - cb * D;
            int cube = pos0 / g.C + cb;
            if (cube < g.N_live) {
                double acc = 0.0;                                   // empty slots hold zeros
                for (int r = 0; r < g.C; ++r) acc += (double)__bfloat162float(Ks[cb * g.C + r][d]);
                cube_keys[((size_t)(b * g.Hkv + gk) * g.N + cube) * D + d] = (float)(acc / (double)cube_tokens_held(g, cube));
            }
        }
    }
}

// Mean keys for cubes of more than 64 tokens: one CTA per (cube, kv head, batch), D threads,
// reading the cube-major keys just written by relayout_pool_kernel.
__global__ void pool_large_cubes_kernel(Geom g, const __nv_bfloat16* __restrict__ k_cube,
                                        float* __restrict__ cube_keys) {
    const int cube = blockIdx.x + (g.pos_begin >> g.c_shift), gk = blockIdx.y, b = blockIdx.z, d = threadIdx.x;
    if (d >= g.D) return;
    const __nv_bfloat16* src = k_cube + ((size_t)(b * g.Hkv + gk) * g.S_cap + (size_t)cube * g.C) * g.D + d;
    // sixteen loads in flight, added in token order (the order of a plain loop: the sum is the same bit for bit)
    double acc = 0.0;
    for (int r0 = 0; r0 < g.C; r0 += 16) {               // C is a multiple of 64 here
        __nv_bfloat16 x[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) x[i] = src[(size_t)(r0 + i) * g.D];
#pragma unroll
        for (int i = 0; i < 16; ++i) acc += (double)__bfloat162float(x[i]);
    }
    cube_keys[((size_t)(b * g.Hkv + gk) * g.N + cube) * g.D + d] = (float)(acc / (double)cube_tokens_held(g, cube));
}

}  // namespace adaspark
