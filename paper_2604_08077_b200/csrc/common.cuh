// Shared device-side definitions for the AdaS-Attn kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace adaspark {

constexpr int kTileRows = 128;  // query rows per tile (cube-major positions)
constexpr int kBlockTok = 64;   // key/value tokens per block (cube-major positions)

// Division of a non-negative int (< 2^31) by a runtime constant without a divide instruction:
// with s = ceil(log2 d) and mul = floor(2^32 * (2^s - d) / d) + 1, n / d = (hi32(n * mul) + n) >> s.
struct FastDiv {
    uint32_t mul, shift;
    int d;
    __host__ void init(int divisor) {
        d = divisor;
        shift = 0;
        while ((1ll << shift) < (long long)divisor) ++shift;
        mul = (uint32_t)((((1ull << shift) - (unsigned long long)divisor) << 32) / (unsigned long long)divisor + 1ull);
    }
    __host__ __device__ __forceinline__ int div(int n) const {
#ifdef __CUDA_ARCH__
        return (int)((__umulhi((uint32_t)n, mul) + (uint32_t)n) >> shift);
#else
        return (int)(((uint32_t)(((unsigned long long)(uint32_t)n * mul) >> 32) + (uint32_t)n) >> shift);
#endif
    }
    __host__ __device__ __forceinline__ void divmod(int n, int& q, int& r) const {
        q = div(n);
        r = n - q * d;
    }
};

// Geometry of one partitioned problem (Sec. 3.1).  "pos" is the cube-major position of a token in
// the caches: the video token of cube c with in-window rank r sits at pos = c*C + r (a cube at the far
// face of a grid that the window does not divide holds fewer tokens than its C slots: the other slots
// stay empty), text token u at S_v + u.  Text that precedes the video in the sequence (a prompt prefix,
// n_prefix tokens) occupies the first n_prefix text slots: it is attended by every video and text row in
// full and is no candidate of Eq. 1; the text after the video follows it.
struct Geom {
    int B, T, H, W;      // batch, frames, patch rows, patch columns
    int ct, ch, cw;      // cube window
    int nH, nW;          // cube grid: H/ch, W/cw
    int C, N;            // tokens per cube (a power of two), cubes
    int c_shift;         // log2(C)
    int cw_shift, ch_shift;   // log2(cw), log2(ch): C is a power of two, so every window side is one
    FastDiv div_nW, div_nH, div_n_tiles, div_Hq;
    int S_v, n_text, S;  // video slots N*C of the partition, text tokens so far (prefix included), slots present after this call
    int S_tok;           // video tokens T*H*W (= S_v unless the grid is ragged)
    int n_prefix;        // text tokens of the sequence that precede the video
    int ragged;          // 1: the window does not divide the grid (some slots of boundary cubes are empty)
    // Row window of this call (chunked prefill): the q/k/v/out tensors hold the S_io tokens whose
    // cube-major positions are [pos_begin, S) -- whole time blocks of cubes, so they are also the raster
    // tokens pos_begin .. -- and only those rows are computed.  One-shot prefill: pos_begin = 0, S_io = S.
    int pos_begin, S_io;
    int frame_begin;     // first frame of this call's tensors
    int N_live;          // cubes present after this call (<= N)
    int tile_begin;      // pos_begin / 128
    int S_cap;           // cache rows per (b, kv head), multiple of 128
    int n_words;         // ceil(N/32)
    int n_tiles;         // ceil(S/128) query tiles of this call
    int n_tiles_cap;     // S_cap/128 (stride of per-tile buffers)
    int n_kv_blocks_cap; // S_cap/64
    int Hq, Hkv, G, D;
    int N_ld;            // leading dimension of the logits scratch (N rounded up to 64)
    float scale;         // logit scale as float (attention softmax)
    float scale_log2;    // scale * log2(e)
    double scale_d;      // logit scale in double (selection scores)
    double top_p;
    int top_k;           // > 0: Top-K rule instead of Top-p
};

// O1 inverse: cube-major position -> index of the token in the sequence [prefix][video, raster][text],
// or -1 for a slot that holds no token.
__device__ __forceinline__ int pos_to_io(const Geom& g, int pos) {
    if (pos >= g.S_v) {
        const int u = pos - g.S_v;
        return u < g.n_prefix ? u : u + g.S_tok;        // text after the video: n_prefix + S_tok + (u - n_prefix)
    }
    const int c = pos >> g.c_shift, r = pos & (g.C - 1);
    int cx, cy, cb, t;
    g.div_nW.divmod(c, t, cx);
    g.div_nH.divmod(t, cb, cy);
    const int rx = r & (g.cw - 1);
    const int ry = (r >> g.cw_shift) & (g.ch - 1);
    const int rt = r >> (g.cw_shift + g.ch_shift);
    const int tt = cb * g.ct + rt, yy = cy * g.ch + ry, xx = cx * g.cw + rx;
    if (g.ragged && (tt >= g.T || yy >= g.H || xx >= g.W)) return -1;
    return g.n_prefix + (tt * g.H + yy) * g.W + xx;
}

// Does the slot at pos hold a token of the sequence so far?
__device__ __forceinline__ bool slot_live(const Geom& g, int pos) {
    return pos < g.S && (!g.ragged || pos >= g.S_v || pos_to_io(g, pos) >= 0);
}

// Row of the call's q/k/v/out tensors (batch b) that holds the token at cube-major position pos (a live slot).
__device__ __forceinline__ size_t io_row(const Geom& g, int b, int pos) {
    return (size_t)b * g.S_io + (pos_to_io(g, pos) - g.pos_begin);
}

// Number of candidate cubes of the row at `pos`: preceding cubes for video, none for the prefix, all cubes
// for the text after the video.
__device__ __forceinline__ int n_candidates(const Geom& g, int pos) {
    return pos < g.S_v ? (pos >> g.c_shift) : (pos < g.S_v + g.n_prefix ? 0 : g.N);
}

// Largest candidate count among the rows of query tile `tile` (candidate counts grow along the video, drop
// to zero on the text prefix and are N on the text after it).
__device__ __forceinline__ int tile_max_candidates(const Geom& g, int tile) {
    const int first = tile * kTileRows, last = min(first + kTileRows, g.S) - 1;
    int m = n_candidates(g, last);
    if (first < g.S_v && last >= g.S_v) m = max(m, n_candidates(g, g.S_v - 1));
    return m;
}

// First 64-key block of the local range of the 256-row pair of query tiles that starts at pair_pos0: the block
// that holds the first slot of the own cube of the pair's first row (video) or the first text slot.  Cubes
// that end before this block are attended only if selected; from this block on the per-key rule applies.
__device__ __forceinline__ int pair_first_local_blk(const Geom& g, int pair_pos0) {
    const int local_start = pair_pos0 < g.S_v ? ((pair_pos0 >> g.c_shift) << g.c_shift) : g.S_v;
    return local_start / kBlockTok;
}

// Per-tile selection mask matrix: word w of row r of global tile gt at
// mask[(gt * n_words + w) * 128 + r]; gt = (b*Hq + h) * n_tiles_cap + tile.
__device__ __forceinline__ size_t mask_index(const Geom& g, int b, int h, int tile, int w, int r) {
    return ((size_t)((b * g.Hq + h) * g.n_tiles_cap + tile) * g.n_words + w) * kTileRows + r;
}

// Key visibility (Eq. 3 + text rule): may the row at cube-major position pr attend the key at pk?
// `word` is the row's selection word that covers cube pk/C (bits of cubes that are not
// candidates of the row are never set by the selection kernel).
__device__ __forceinline__ bool key_allowed(const Geom& g, int pr, int pk, uint32_t word) {
    if (pk >= g.S_v) return pk <= pr || (pr < g.S_v && pk < g.S_v + g.n_prefix);   // text causally; the prefix for every video row
    if (g.ragged && pos_to_io(g, pk) < 0) return false;                            // an empty slot of a boundary cube
    if (pk <= pr && (pk >> g.c_shift) == (pr >> g.c_shift)) return true;           // own cube up to the query
    return (word >> ((pk >> g.c_shift) & 31)) & 1u;                                // selected cube
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void cp_async_16(void* smem_dst, const void* gmem_src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(smem_u32(smem_dst)),
                 "l"(gmem_src));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                            const void* smem_ptr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(smem_u32(smem_ptr)));
}

// D = A(16x16, row) * B(16x8, col) + D, bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                               uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// D = A(8x4, row) * B(4x8, col) + D in fp64.
__device__ __forceinline__ void mma_f64_884(double (&d)[2], double a, double b) {
    asm volatile(
        "mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};\n"
        : "+d"(d[0]), "+d"(d[1])
        : "d"(a), "d"(b));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// 2^x on the FMA pipe, for part of a softmax row's exponentials when the MUFU unit (4 lanes per
// scheduler: 8 cycles per warp instruction) is the busier pipe.  x = n + f with n = round(x), f in
// [-0.5, 0.5]: a cubic for 2^f (minimax in relative error over that interval, 7.7e-5: far inside the
// bf16 rounding of the probabilities it feeds), n added to the exponent field.  x is clamped at -125,
// so a masked score (-inf) yields about 2^-125 = 2e-38 instead of 0: next to any visible key (weight
// >= 2^-8 of the row's reference) that is nothing in an fp32 sum, and it is multiplied by 0 when the
// row meets its first visible key.  (An exact zero costs one more instruction per element, which
// measurably undoes the gain.)
__device__ __forceinline__ float fma_exp2(float x) {
    const float xc = fmaxf(x, -125.f);
    const float xr = xc + 12582912.f;                  // 1.5 * 2^23: the low mantissa bits now hold n
    const float f = xc - (xr - 12582912.f);
    const float p = fmaf(fmaf(fmaf(0.055222616f, f, 0.24261537f), f, 0.69325161f), f, 0.99992758f);
    return __uint_as_float(__float_as_uint(p) + (__float_as_uint(xr) << 23));
}

// ---- packed fp32 pairs (sm_100): one instruction for two lanes of a*b+c / a+b -------------------
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
    unsigned long long d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "r"(__float_as_uint(lo)), "r"(__float_as_uint(hi)));
    return d;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
    uint32_t a, b;
    asm("mov.b64 {%0, %1}, %2;" : "=r"(a), "=r"(b) : "l"(v));
    lo = __uint_as_float(a);
    hi = __uint_as_float(b);
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long add_f32x2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// byte offset of 16-byte chunk `chunk` of 128-byte row `row` under the 128-byte swizzle
__device__ __forceinline__ int sw128(int row, int chunk) { return row * 128 + ((chunk ^ (row & 7)) << 4); }

// ---- sm_100 three-input float maximum ------------------------------------------
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

}  // namespace adaspark
