/*
 * adaspark_attn.h - C ABI of the B200 (sm_100a) implementation of Adaptive Cube-Selective
 * Attention (AdaS-Attn; Sec. 3.1-3.2 and Algorithm 1 of the AdaSpark paper).
 *
 * The library computes, for a sequence laid out as [video tokens (T x H x W raster)][text tokens]:
 *   1. the cube partition of the video tokens by a (cube_t, cube_h, cube_w) window and the
 *      cube-major re-layout of K and V                       (Sec. 3.1; Algorithm 1, "Reshape K,V");
 *   2. one mean key per cube and KV head                      (Sec. 3.2, definition under Eq. 1);
 *   3. for every query row the softmax over the scaled scores against the mean keys of its
 *      candidate cubes (the preceding cubes for a video query, all cubes for a text query)
 *                                                             (Eq. 1; text rule after Eq. 3);
 *   4. the nucleus (Top-p) cube set: the shortest prefix of the cubes sorted by probability
 *      (descending; equal probabilities by lower cube index) whose mass reaches top_p (Eq. 2);
 *   5. one softmax attention over the tokens of the selected cubes plus the causal prefix of
 *      the query's own cube (video) or of the text (text), written back in raster order
 *                                                             (Eq. 3; Algorithm 1, "Restore").
 * A decode step evaluates one new text token per sequence against caches built by the prefill.
 *
 * Conventions
 *   - All tensor pointers are DEVICE pointers owned by the caller; the library never allocates
 *     device memory in _forward / _decode and never synchronises the host with the device.
 *     Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*; NULL = default stream).
 *   - Tensors are bf16, row-major, raster order: q/out [B,S,Hq,D], k/v [B,S,Hkv,D] with
 *     S = T*H*W + n_text and video token (t,y,x) at s = (t*H + y)*W + x (after the n_prefix prefix
 *     tokens of adaspark_attn_forward_prefix).  Q and K are post-RoPE.
 *   - Query head h uses KV head h / (Hq/Hkv).  Mean keys are per KV head, selection per query head.
 *   - Errors are return codes; argument errors are found on the host before any launch.
 *     adaspark_attn_last_error() returns a message for the most recent failure on a handle.
 *   - No CPU fallback exists: without a CUDA device every compute entry point fails.
 */
#ifndef ADASPARK_ATTN_H_
#define ADASPARK_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct adaspark_attn adaspark_attn_t; /* opaque, library-owned */

typedef enum {
    ADASPARK_OK = 0,
    ADASPARK_ERR_INVALID_ARG = 1,
    ADASPARK_ERR_UNSUPPORTED = 2,
    ADASPARK_ERR_NOT_PARTITIONED = 3,
    ADASPARK_ERR_WORKSPACE_TOO_SMALL = 4,
    ADASPARK_ERR_CUDA = 5,
    ADASPARK_ERR_TIMEOUT = 6
} adaspark_status_t;

/* Problem statement of Algorithm 1: cube window, heads, head_dim, nucleus mass p. */
typedef struct {
    int32_t cube_t, cube_h, cube_w; /* cube window in frames / patch rows / patch columns     */
    int32_t n_q_heads, n_kv_heads;  /* n_kv_heads must divide n_q_heads (GQA group size <= 16) */
    int32_t head_dim;               /* 64 or 128                                               */
    float top_p;                    /* in (0, 1]; >= 1 selects every candidate cube (dense)    */
    float softmax_scale;            /* 0 => 1/sqrt(head_dim) (Eqs. 1, 3); used for both        */
    int32_t device;                 /* CUDA ordinal                                            */
    int32_t top_k;                  /* 0: Top-p (Eq. 2).  > 0: keep the top_k most probable
                                       candidate cubes instead (all of them if fewer exist), the
                                       fixed-budget rule of the paper's selection ablation;
                                       top_p is then ignored                                    */
} adaspark_attn_config_t;

/* Sizes fixed by _partition.  "pos" below is the cube-major position of a token:
 * pos = cube * cube_tokens + rank for video tokens, s_video + u for text token u. */
typedef struct {
    int64_t n_cubes;         /* N                                                              */
    int64_t cube_tokens;     /* C = cube_t*cube_h*cube_w                                       */
    int64_t s_video;         /* video slots N*C (= T*H*W when the cube window divides the grid) */
    int64_t s_cap;           /* cache rows per (batch, kv head): s_video + n_text_max + 1
                                rounded up to a multiple of 128                                */
    int64_t bitmap_words;    /* ceil(N/32): uint32 words per selection bitmap row              */
    int64_t k_cube_bytes;    /* bf16 [B, Hkv, s_cap, D]: keys at cube-major positions          */
    int64_t v_cube_bytes;    /* bf16 [B, Hkv, s_cap/64, D, 64]: per 64-position block, V^T     */
    int64_t cube_keys_bytes; /* fp32 [B, Hkv, N, D]: mean keys                                 */
    int64_t forward_workspace_bytes;
    int64_t decode_workspace_bytes;
} adaspark_attn_layout_t;

/* Header the library keeps in the first bytes of the workspace of _forward / _decode.  It is
 * reset at the start of every call; the caller may copy it to the host after synchronising. */
typedef struct {
    int32_t status;               /* 0 = ok; 1 = text_len out of range (decode); 6 = a bounded
                                     device wait expired (ADASPARK_ERR_TIMEOUT)               */
    int32_t reserved;
    uint64_t executed_kv_blocks;  /* prefill: (128 query rows, 64-key block) products the attention
                                     kernels computed (union path: per tile and visited block;
                                     gather path: per item); executed FLOPs = this * 128*64*D*4 */
    uint64_t decode_kv_blocks;    /* decode: 64-key blocks gathered, summed over (b, kv head) */
    uint32_t fallback_rows;       /* prefill: query rows whose selection the tensor-core kernel
                                     left to the fp64 selection kernel (normally 0)           */
    uint32_t max_tile_kv_blocks;  /* prefill: largest number of 64-key blocks one 256-row pair of
                                     query tiles visited (load imbalance: compare with the mean
                                     executed_kv_blocks / 2 / number of pair tiles)           */
    uint32_t gather_entries;      /* prefill: (query row, 64-key block) entries computed by the
                                     query-gather path (0: every pair took the union path)     */
    uint32_t gather_items;        /* ... in this many items of up to 128 gathered rows          */
    uint32_t gather_pair_tiles;   /* ... for this many 256-row pairs of query tiles             */
    uint32_t reserved2;
} adaspark_attn_workspace_header_t;

/* Create a handle for one configuration.  Host only.  Fails with ERR_UNSUPPORTED for a
 * head_dim other than 64/128, a cube window whose token count C is not one of
 * {16, 32, 64, 128, 256, 512, 1024}, or a GQA group size above 16; with ERR_INVALID_ARG for
 * non-positive sizes, top_p <= 0, top_k < 0, or a NULL pointer. */
adaspark_status_t adaspark_attn_create(const adaspark_attn_config_t *config,
                                       adaspark_attn_t **out_handle);

/* Sec. 3.1: fix the video grid and derive the cube partition (N cubes of C tokens) and every
 * buffer size.  `batch`, `frames`, `grid_h`, `grid_w` describe the video token grid;
 * `n_text_max` is the largest number of text tokens any later _forward/_decode will hold.
 * `*workspace_bytes` (nullable) receives max(forward, decode) workspace size.  Host only.
 * A grid the cube window does not divide (the paper is silent) is covered by ceil(T/cube_t) x
 * ceil(H/cube_h) x ceil(W/cube_w) cubes: the cubes at the far faces hold fewer tokens, their mean key is
 * the mean over the tokens they hold, their other slots stay empty in the caches and are never attended.
 * ERR_UNSUPPORTED if N > 4096 or the cache would hold more than 2097152 rows per sequence
 * (s_video + n_text_max + 1).
 * The forward workspace holds the selection masks, the digit planes of the mean keys and the buffers of the
 * query-gather path; cube scores are never stored and Q is read where the caller left it. */
adaspark_status_t adaspark_attn_partition(adaspark_attn_t *handle, int32_t batch, int32_t frames,
                                          int32_t grid_h, int32_t grid_w, int32_t n_text_max,
                                          size_t *workspace_bytes);

/* Sizes derived by the last _partition.  ERR_NOT_PARTITIONED before it. */
adaspark_status_t adaspark_attn_get_layout(const adaspark_attn_t *handle,
                                           adaspark_attn_layout_t *out_layout);

/* Prefill (Algorithm 1, the AdaS-Attn lines; Eqs. 1-3).
 *   q, k, v      in : bf16 [B, S, H*, D] raster, S = s_video + n_text, 0 <= n_text <= n_text_max.
 *                     q and out may both be NULL: then only the caches are built.
 *   out          out: bf16 [B, S, Hq, D] raster.
 *   k_cube, v_cube, cube_keys
 *                out: the caches described in adaspark_attn_layout_t (caller-allocated, written
 *                     in full; rows beyond S are zero-filled).
 *   sel_bitmap   out, nullable: uint32 [B, Hq, S, bitmap_words], bit j of a row (raster token
 *                     order) is set iff cube j is in the row's nucleus S_i.
 *   sel_count    out, nullable: int32 [B, Hq, S] = |S_i|.
 *   workspace    device scratch of at least forward_workspace_bytes, 256-byte aligned.
 * Enqueues its kernels on `cuda_stream` and returns; no host synchronisation, no other stream, no
 * allocation.  The Q tiles of the attention kernel are TMA boxes of `q` itself (the tensor map is built
 * on the host per call): `q` needs 16-byte alignment and must stay valid until the call's work is done.
 * Which of the two attention paths a pair of query tiles takes (union of the selected key blocks, or
 * the query-gather path of adaspark_attn_set_gather) is decided on the device; the workspace header
 * reports it. */
adaspark_status_t adaspark_attn_forward(adaspark_attn_t *handle, const void *q, const void *k,
                                        const void *v, int32_t n_text, void *out, void *k_cube,
                                        void *v_cube, float *cube_keys, uint32_t *sel_bitmap,
                                        int32_t *sel_count, void *workspace,
                                        size_t workspace_bytes, void *cuda_stream);

/* Prefill of a sequence whose text partly PRECEDES the video: [n_prefix text tokens][video][n_text
 * text tokens] (the paper places the text after the video and is silent on a prompt before it).
 * Reading taken: the prefix is attended by every video and text token always and in full, like a
 * token's own cube: it is no candidate of Eq. 1, its mass does not count toward top_p, and prefix
 * tokens attend causally among themselves.  q/k/v/out hold the n_prefix + T*H*W + n_text tokens in
 * that order; n_prefix + n_text <= n_text_max.  In the caches the prefix occupies the first n_prefix
 * text slots (positions s_video ..), the later text follows it; a decode step after it passes
 * text_len = n_prefix + n_text.  Everything else as adaspark_attn_forward (= n_prefix 0). */
adaspark_status_t adaspark_attn_forward_prefix(adaspark_attn_t *handle, const void *q, const void *k,
                                               const void *v, int32_t n_prefix, int32_t n_text,
                                               void *out, void *k_cube, void *v_cube,
                                               float *cube_keys, uint32_t *sel_bitmap,
                                               int32_t *sel_count, void *workspace,
                                               size_t workspace_bytes, void *cuda_stream);

/* adaspark_attn_forward with HOST input and output buffers: the call copies q, k, v from host memory
 * into the caller's device buffers, runs the prefill there and copies `out` back, all enqueued on
 * `cuda_stream` (no host synchronisation: the output is in out_host once the stream has reached
 * this point; use pinned host memory for the copies to be asynchronous).
 *   q_host, k_host, v_host  in : host bf16 [B, S, H*, D] as in adaspark_attn_forward (q_host and
 *                                out_host may both be NULL: caches only).
 *   out_host                out: host bf16 [B, S, Hq, D].
 *   q_dev, k_dev, v_dev, out_dev  caller-owned DEVICE staging buffers of the same shapes (the
 *                                library allocates nothing); their contents are overwritten.
 * Everything else as adaspark_attn_forward. */
adaspark_status_t adaspark_attn_forward_host(adaspark_attn_t *handle, const void *q_host,
                                             const void *k_host, const void *v_host, int32_t n_text,
                                             void *out_host, void *q_dev, void *k_dev, void *v_dev,
                                             void *out_dev, void *k_cube, void *v_cube,
                                             float *cube_keys, void *workspace,
                                             size_t workspace_bytes, void *cuda_stream);

/* Chunked prefill: the same computation as adaspark_attn_forward, fed one run of frames at a time
 * (the long-video setting of the paper: a later frame never changes an earlier row, because a video
 * query of Eq. 1 only sees the cubes that precede its own and the text comes after the video).
 * The call brings frames [frame_begin, frame_begin + frame_count) of every sequence: it appends
 * their cubes to k_cube / v_cube / cube_keys and computes `out` for these tokens only, attending the
 * cubes of earlier calls through the caches.
 *   frame_begin, frame_count  multiples of cube_t (whole time blocks of cubes); frame_begin * H * W
 *                must be a multiple of 256 (ERR_UNSUPPORTED otherwise; so is a grid that the cube
 *                window does not divide, except through the single chunk (0, T)).  Chunks must be fed in
 *                order, without gaps, to the same caches; the library keeps no record of them.
 *   n_text       < 0: more video follows (no text in this call).  >= 0: this is the last call of the
 *                sequence: it must end the video (frame_begin + frame_count = T; frame_count may be 0
 *                when the video is already complete), brings n_text text tokens after its frames,
 *                and zero-fills the caches beyond the sequence up to their capacity.
 *   q, k, v, out bf16 [B, frame_count*H*W + max(n_text, 0), H*, D]: this call's tokens in raster order
 *                (then its text tokens).  q and out may both be NULL (caches only).
 *   sel_bitmap / sel_count  nullable, rows of this call only: [B, Hq, tokens of the call, ...].
 * Everything else as adaspark_attn_forward; adaspark_attn_forward(n_text) is the single chunk
 * (0, T, n_text).  The selection is the same bit for bit however the frames are cut; outputs agree within the
 * bf16 rounding of the attention weights (a call that starts at frame 0 may fix a row's softmax reference in
 * advance from the norms of the keys it brought, a later call uses the running maximum). */
adaspark_status_t adaspark_attn_forward_chunk(adaspark_attn_t *handle, const void *q, const void *k,
                                              const void *v, int32_t frame_begin, int32_t frame_count,
                                              int32_t n_text, void *out, void *k_cube, void *v_cube,
                                              float *cube_keys, uint32_t *sel_bitmap,
                                              int32_t *sel_count, void *workspace,
                                              size_t workspace_bytes, void *cuda_stream);

/* Decode: one new text token per sequence (the text-token rule after Eq. 3 applied to a row
 * appended after the cached sequence; the new token attends itself).
 *   q_new        in : bf16 [B, 1, Hq, D].
 *   k_new, v_new in : bf16 [B, 1, Hkv, D]; written into the caches at text slot text_len[b].
 *                     Both may be NULL when the caller has already stored the new token's K/V
 *                     in slot text_len[b] of the caches.
 *   k_cube, v_cube  in/out, cube_keys in: caches written by _forward.
 *   text_len     in : device int32 [B], text tokens cached before this step, 0 <= text_len[b]
 *                     <= n_text_max.  The row attends text slots 0..text_len[b] (itself included).
 *                     A value outside that range (checked on the device, with or without k_new)
 *                     sets `status` in the workspace header to 1, writes nothing to the caches
 *                     and yields a zero output row for that sequence.
 *   out          out: bf16 [B, 1, Hq, D].
 *   sel_bitmap   out, nullable: uint32 [B, Hq, bitmap_words].
 *   workspace    device scratch of at least decode_workspace_bytes, 256-byte aligned. */
adaspark_status_t adaspark_attn_decode(adaspark_attn_t *handle, const void *q_new,
                                       const void *k_new, const void *v_new, void *k_cube,
                                       void *v_cube, const float *cube_keys,
                                       const int32_t *text_len, void *out, uint32_t *sel_bitmap,
                                       void *workspace, size_t workspace_bytes,
                                       void *cuda_stream);

/* Bytes of decode scratch built into the library image (see adaspark_attn_decode_static). */
#define ADASPARK_ATTN_STATIC_SCRATCH_BYTES (8u << 20)

/* adaspark_attn_decode without a workspace argument.  (The paper has no counterpart: this entry
 * point exists only for the convenience of some callers.)
 *
 * It is meant for callers that have no way to allocate device memory at the moment they decode:
 * a serving process that has handed all of the GPU's memory to its own pool and cannot carve a
 * workspace out of it for a foreign library, or a latency-critical decode loop in which a
 * cudaMalloc (which may block on all outstanding work of the device) is not acceptable.  Such a
 * caller passes only the inputs, caches and the output; the split-KV partials, block lists and
 * bitmaps go to a fixed array of ADASPARK_ATTN_STATIC_SCRATCH_BYTES (8 MiB) that is part of the
 * library itself.  Every GPU on which the library is loaded holds that array until the process
 * exits, whether or not this call is ever used.
 *
 * Arguments, results and errors are those of adaspark_attn_decode.  In addition:
 *   - ERR_WORKSPACE_TOO_SMALL if the partition's decode_workspace_bytes exceeds the 8 MiB
 *     (a 131072-token video cache in 2048 cubes with 28/4 heads of 128 fits up to batch 8; at batch 16
 *     it needs about 10 MiB); use adaspark_attn_decode then.
 *   - The first call on each device looks up the array's device address (a one-time host-side
 *     set-up with that device current); make that first call before any stream capture begins.
 *     The address is cached for the life of the process and is valid only while the device's
 *     primary context lives: after a cudaDeviceReset by the host program it is stale, and this
 *     entry point must not be called again in that process.
 *   - The call performs no cudaMalloc / cudaFree and uses no allocating library routine.
 *   - All calls on a device share the one array, which keeps whatever the previous call left in
 *     it; the header that must start at zero is cleared by every call.  Two calls whose kernels
 *     may overlap on the GPU (different streams, or different handles on the same device) race
 *     on the array: serialise them. */
adaspark_status_t adaspark_attn_decode_static(adaspark_attn_t *handle, const void *q_new,
                                              const void *k_new, const void *v_new, void *k_cube,
                                              void *v_cube, const float *cube_keys,
                                              const int32_t *text_len, void *out,
                                              uint32_t *sel_bitmap, void *cuda_stream);

/* Release the handle: its host memory and, if stage timing was enabled, the timing events.  It does
 * not wait for work enqueued on the caller's streams, and the caller's buffers are not touched: destroy
 * the handle after that work is done.  NULL is accepted. */
adaspark_status_t adaspark_attn_destroy(adaspark_attn_t *handle);

/* Message of the most recent error on this handle ("" if none). Never NULL. */
const char *adaspark_attn_last_error(const adaspark_attn_t *handle);

/* Number of kernel launches the most recent _forward / _decode enqueued (host counter). */
int64_t adaspark_attn_last_launch_count(const adaspark_attn_t *handle);

/* Stage timing for measurement: when enabled, _forward / _decode record CUDA events on the
 * caller's stream around their stages.  adaspark_attn_get_stage_times waits for the last
 * recorded event (the only host synchronisation in the library, and only in this call) and
 * returns milliseconds: prefill {re-layout+pooling, scoring+selection, attention, 0};
 * decode {0, append+scoring+selection+plan, split-KV attention, combine} (the append of the new
 * token is fused into the selection kernel). */
adaspark_status_t adaspark_attn_enable_stage_timing(adaspark_attn_t *handle, int32_t enable);
adaspark_status_t adaspark_attn_get_stage_times(adaspark_attn_t *handle, float *ms_out /* host [4] */);
/* With stage timing on, the last prefill's union attention kernel alone (Eq. 3 on the tensor cores, kernels
 * 1 and 2), in milliseconds: the attention stage also holds the small kernels of the query-gather decision.
 * Waits for that kernel's end event.  ERR_INVALID_ARG if no timed tcgen05 prefill was recorded. */
adaspark_status_t adaspark_attn_get_attention_kernel_ms(adaspark_attn_t *handle, float *ms_out /* host [1] */);

/* Selects the prefill kernels: 0 = mma.sync attention + fp64 (mma.m8n8k4.f64) scoring, the legacy
 * tensor path kept as a cross-check; 1 = tcgen05/TMEM attention with TMA-staged tiles + tcgen05
 * scoring from error-free digit slices (default when built in); 2 = tcgen05 attention + fp64
 * scoring.  ERR_UNSUPPORTED for an unknown value. */
adaspark_status_t adaspark_attn_set_prefill_kernel(adaspark_attn_t *handle, int32_t which);

/* Query-gather path of the prefill (kernels 1 only; Eq. 3 over the selected cubes alone).  The attention
 * kernel visits, per pair of 128-row query tiles, the union of the key blocks its 256 rows selected; when
 * the rows pick different cubes that union is nearly every block.  For such pairs the library instead
 * gathers, per 64-key block, the query rows (of all tiles and all heads of the GQA group) that selected a
 * cube in it, computes their attention over that block on the tensor cores, and merges each row's partial
 * results with the result of its local range (own cube, text) by the softmax identity.  The choice is made
 * on the device, per pair: gathered iff (row, key block) entries of the pair's rows <= pairs_per_block *
 * key blocks in the pair's union -- and only if all qualifying pairs together save more than the fixed
 * cost of the path (about 50 us by the library's estimate, in which a union block costs as much as 44
 * entries).  pairs_per_block = 0 switches the path off (every pair takes the union path); a value above 44
 * forces it for every pair that meets the threshold, a huge value for every pair with a selected cube.  budget_bytes bounds the workspace
 * the path may use for its partial results (2*head_dim + 24 bytes per entry; _partition reserves
 * min(budget, pairs_per_block * video key blocks / 512 entries per query row -- what the pairs of a causal
 * sequence can produce on average --, 128 entries per query row));
 * if the pairs that qualify in a call need more, only part of them is gathered in that call: the pairs fall
 * into four classes by entries per union block (up to 1/8, 1/4, 1/2 of the threshold, up to the threshold)
 * and into row windows; (class, window) units are kept while they fit, sparsest class first and inside a
 * class the latest rows first.  Budget and
 * threshold size the forward workspace: set them before _partition (a different budget afterwards is
 * ERR_INVALID_ARG; the threshold may still change, the reserved capacity does not).  Defaults: 30 entries
 * per block (gathering pays up to about 44 on a B200), 24 GiB.  Outputs agree with the union path within
 * bf16 rounding of the partial results; the selection is the same. */
adaspark_status_t adaspark_attn_set_gather(adaspark_attn_t *handle, float pairs_per_block,
                                           uint64_t budget_bytes);

#ifdef __cplusplus
}
#endif
#endif /* ADASPARK_ATTN_H_ */
