/*
 * AdaS-Attn oracle: a plain, slow, fp64 CPU statement of Adaptive Cube-Selective Attention.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product path may call this file; it shares no
 * code with the CUDA implementation.  It follows the paper's definitions step by step, with
 * no blocking, fusion or reordering:
 *
 *   O1  cube partition / cube-major order        Sec. 3.1; Algorithm 1 ("Reshape K,V into Cubes")
 *   O2  mean key per cube and KV head            Sec. 3.2, text under Eq. 1
 *   O3  selection scores + softmax over cubes    Eq. 1
 *   O4  nucleus (Top-p) cube selection           Eq. 2
 *   O4k Top-K cube selection (the fixed-budget rule the paper compares Top-p with in its
 *       selection-strategy ablation): the K most probable candidate cubes
 *   O5  attention over selected cubes + own-cube Eq. 3 and the text-token rule that follows it
 *       prefix (video) or text prefix (text)
 *   O6  decode = a text-rule row appended after the cached sequence (same code as O5)
 *
 * Readings taken where the paper is silent (each also listed in the design notes):
 *   - a query attends itself (standard causal "<="), otherwise p = 1 would not be dense
 *     causal attention;
 *   - cubes are numbered row-major over (time block, row block, column block), tokens inside
 *     a cube row-major over (t, y, x); "preceding" refers to this cube-major order;
 *   - Top-p = the shortest prefix of the cubes sorted by (probability descending, index
 *     ascending) whose cumulative probability is >= p; p >= 1 selects every candidate;
 *   - the own cube is never a candidate; text queries see every video cube as a candidate;
 *   - with grouped-query attention the mean keys are per KV head, the selection per query
 *     head (kv head = query head / group size);
 *   - a video grid that the cube window does not divide is covered by ceil(T/ct) x ceil(H/ch) x
 *     ceil(W/cw) cubes; the cubes at the far faces hold fewer tokens, their mean key is the mean
 *     over the tokens they do hold, and only those tokens are attended when the cube is selected;
 *   - text placed BEFORE the video (a prompt prefix; n_prefix tokens) is attended by every later
 *     token always and in full, like the own cube: it is never a candidate of Eq. 1 and its
 *     mass does not count toward p; prefix tokens themselves attend causally among themselves.
 *
 * Pins (tests/test_oracle_*.py): closed-form permutation examples, numpy reshape-mean,
 * brute force over all cube subsets, p -> 0 argmax, p = 1 equals an independently written
 * dense causal attention, first-cube special case, equal-keys error bound, V-linearity,
 * logit-shift invariance.  The paper prints no worked numeric example, so absolute output
 * values are pinned only through those identities.
 *
 * All tensors are raster order, row-major:  Q [B,S,Hq,D], K,V [B,S,Hkv,D] as float (the
 * bf16-rounded inputs widened exactly), S = n_prefix + T*H*W + n_text: prefix text, video
 * tokens (t, y, x) row-major, text.
 *
 * "Position" below is the place of a token in the causal order: prefix token u at u, the video
 * token of cube c with in-window rank r at n_prefix + c*C + r (slots of a boundary cube that
 * fall outside the grid hold no token), text token u at n_prefix + N*C + u.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int32_t B, T, H, W;      /* batch, frames, patch rows, patch columns              */
    int32_t ct, ch, cw;      /* cube window                                           */
    int32_t n_text;          /* text tokens after the video                           */
    int32_t Hq, Hkv, D;      /* query heads, KV heads, head dim                       */
    double top_p;            /* nucleus mass p                                        */
    double scale;            /* logit scale, 1/sqrt(D) in the paper                   */
    int32_t top_k;           /* > 0: keep the K most probable cubes instead of Top-p  */
    int32_t n_prefix;        /* text tokens before the video                          */
} adas_shape;

static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static int64_t n_cubes(const adas_shape *s) {
    return ceil_div(s->T, s->ct) * ceil_div(s->H, s->ch) * ceil_div(s->W, s->cw);
}
static int64_t cube_tokens(const adas_shape *s) { return (int64_t)s->ct * s->ch * s->cw; }
static int64_t video_tokens(const adas_shape *s) { return (int64_t)s->T * s->H * s->W; }
static int64_t seq_len(const adas_shape *s) { return s->n_prefix + video_tokens(s) + s->n_text; }
/* number of positions (slots of the causal order, including the empty slots of boundary cubes) */
static int64_t n_positions(const adas_shape *s) { return s->n_prefix + n_cubes(s) * cube_tokens(s) + s->n_text; }
int64_t adas_oracle_num_positions(const adas_shape *s) { return n_positions(s); }

int64_t adas_oracle_num_cubes(const adas_shape *s) { return n_cubes(s); }

/* O1 (Sec. 3.1): token n of the sequence -> its position.  Video token (t, y, x), raster index
 * (t*H + y)*W + x after the prefix, lies in cube ((t/ct)*nH + y/ch)*nW + x/cw with rank
 * ((t%ct)*ch + y%ch)*cw + x%cw. */
int64_t adas_oracle_position(const adas_shape *s, int64_t n) {
    int64_t Sv = video_tokens(s);
    if (n < s->n_prefix) return n;
    n -= s->n_prefix;
    if (n >= Sv) return s->n_prefix + n_cubes(s) * cube_tokens(s) + (n - Sv);
    int64_t x = n % s->W, y = (n / s->W) % s->H, t = n / ((int64_t)s->W * s->H);
    int64_t cube = ((t / s->ct) * ceil_div(s->H, s->ch) + y / s->ch) * ceil_div(s->W, s->cw) + x / s->cw;
    int64_t rank = ((t % s->ct) * s->ch + y % s->ch) * s->cw + x % s->cw;
    return s->n_prefix + cube * cube_tokens(s) + rank;
}

/* pos_of_raster[n] (length S) and its inverse raster_of_pos[pos] (length adas_oracle_num_positions,
 * -1 at the slots that hold no token). */
void adas_oracle_positions(const adas_shape *s, int64_t *pos_of_raster, int64_t *raster_of_pos) {
    int64_t S = seq_len(s), P = n_positions(s);
    for (int64_t p = 0; p < P; ++p) raster_of_pos[p] = -1;
    for (int64_t n = 0; n < S; ++n) {
        int64_t pos = adas_oracle_position(s, n);
        pos_of_raster[n] = pos;
        raster_of_pos[pos] = n;
    }
}

/* O2: kbar[b][g][c][:] = mean of the keys of the tokens of cube c (KV head g): C of them, fewer in
 * a boundary cube of a grid the window does not divide.  kbar: [B,Hkv,N,D]. */
void adas_oracle_mean_keys(const adas_shape *s, const float *K, double *kbar) {
    int64_t S = seq_len(s), Sv = video_tokens(s), N = n_cubes(s), C = cube_tokens(s);
    int64_t D = s->D, Hkv = s->Hkv;
    int64_t *held = (int64_t *)calloc((size_t)N, sizeof(int64_t));
    memset(kbar, 0, sizeof(double) * (size_t)(s->B * Hkv * N * D));
    for (int64_t n = 0; n < Sv; ++n) held[(adas_oracle_position(s, s->n_prefix + n) - s->n_prefix) / C] += 1;
    for (int64_t b = 0; b < s->B; ++b)
        for (int64_t n = 0; n < Sv; ++n) {
            int64_t c = (adas_oracle_position(s, s->n_prefix + n) - s->n_prefix) / C;
            for (int64_t g = 0; g < Hkv; ++g) {
                const float *k = K + ((b * S + s->n_prefix + n) * Hkv + g) * D;
                double *m = kbar + ((b * Hkv + g) * N + c) * D;
                for (int64_t d = 0; d < D; ++d) m[d] += (double)k[d];
            }
        }
    for (int64_t b = 0; b < s->B * Hkv; ++b)
        for (int64_t c = 0; c < N; ++c)
            for (int64_t d = 0; d < D; ++d) kbar[(b * N + c) * D + d] /= (double)held[c];
    free(held);
}

typedef struct { double p; int64_t j; } prob_idx;

static int by_prob_desc_then_index(const void *a, const void *b) {
    const prob_idx *x = (const prob_idx *)a, *y = (const prob_idx *)b;
    if (x->p > y->p) return -1;
    if (x->p < y->p) return 1;
    return (x->j > y->j) - (x->j < y->j);
}

/* O3 + O4 for one query row.
 *   q       [D] query (float), kbar_g [N][D] mean keys of its KV head
 *   n_cand  number of candidate cubes J = {0..n_cand-1}
 * Outputs: sel[j] in {0,1} for j < n_cand (caller zeroes beyond), returns |S|.
 *   probs   (nullable) [n_cand] the softmax P
 *   margin  (nullable) tie margin of the row: min(|c_k* - p|, |c_(k*-1) - p|,
 *           p_(k*) - p_(k*+1)); +inf when nothing can tie (no candidates, or p >= 1).
 *   top_k   > 0: Top-K rule instead of Eq. 2: the first min(K, n_cand) cubes of the same order
 *           (probability descending, index ascending); margin = p_(K) - p_(K+1). */
int64_t adas_oracle_select_row(const float *q, const double *kbar_g, int64_t n_cand, int64_t D,
                               double scale, double top_p, int64_t top_k, uint8_t *sel, double *probs,
                               double *margin) {
    if (margin) *margin = INFINITY;
    if (n_cand <= 0) return 0;
    double *logit = (double *)malloc(sizeof(double) * (size_t)n_cand);
    prob_idx *order = (prob_idx *)malloc(sizeof(prob_idx) * (size_t)n_cand);
    /* Eq. 1: s_j = <q, kbar_j> / sqrt(d_k), P = softmax(s) */
    double mx = -INFINITY;
    for (int64_t j = 0; j < n_cand; ++j) {
        double acc = 0.0;
        for (int64_t d = 0; d < D; ++d) acc += (double)q[d] * kbar_g[j * D + d];
        logit[j] = acc * scale;
        if (logit[j] > mx) mx = logit[j];
    }
    double Z = 0.0;
    for (int64_t j = 0; j < n_cand; ++j) Z += exp(logit[j] - mx);
    for (int64_t j = 0; j < n_cand; ++j) {
        order[j].p = exp(logit[j] - mx) / Z;
        order[j].j = j;
        if (probs) probs[j] = order[j].p;
    }
    /* Eq. 2: nucleus = shortest sorted prefix with cumulative mass >= p */
    qsort(order, (size_t)n_cand, sizeof(prob_idx), by_prob_desc_then_index);
    int64_t kstar = n_cand;
    double cum = 0.0, cum_before = 0.0;
    if (top_k > 0) {
        kstar = top_k < n_cand ? top_k : n_cand;
        if (margin && kstar < n_cand) *margin = order[kstar - 1].p - order[kstar].p;
    } else if (top_p < 1.0) {
        for (int64_t k = 0; k < n_cand; ++k) {
            double before = cum;
            cum += order[k].p;
            if (cum >= top_p) {
                kstar = k + 1;
                cum_before = before;
                break;
            }
        }
        if (margin && kstar <= n_cand && cum >= top_p) {
            double m = fabs(cum - top_p);
            if (fabs(cum_before - top_p) < m) m = fabs(cum_before - top_p);
            if (kstar < n_cand) {
                double gap = order[kstar - 1].p - order[kstar].p;
                if (gap < m) m = gap;
            }
            *margin = m;
        }
    }
    for (int64_t j = 0; j < n_cand; ++j) sel[j] = 0;
    for (int64_t k = 0; k < kstar; ++k) sel[order[k].j] = 1;
    free(logit);
    free(order);
    return kstar;
}

/* O5 for one row whose selection is known.  Key set A = every prefix token (a prefix row: those
 * up to itself), all tokens of every selected cube, plus (video) the own-cube tokens at positions
 * <= the query's, or (text) the text tokens <= the query's.  One softmax over A (Eq. 3), output
 * [D] in fp64.  Returns |A|. */
static int64_t attend_row(const adas_shape *s, const float *Q, const float *K, const float *V,
                          const int64_t *raster_of_pos, int64_t b, int64_t h, int64_t n_raster,
                          int64_t pos, const uint8_t *sel, int64_t n_cand, double *out) {
    int64_t S = seq_len(s), N = n_cubes(s), C = cube_tokens(s), D = s->D, P0 = s->n_prefix;
    int64_t vid_end = P0 + N * C;                       /* first text position */
    int64_t g = h / (s->Hq / s->Hkv);
    const float *q = Q + ((b * S + n_raster) * s->Hq + h) * D;
    /* gather the positions of A (slots without a token are skipped) */
    int64_t cap = P0 + n_cand * C + C + s->n_text + 1, na = 0;
    int64_t *att = (int64_t *)malloc(sizeof(int64_t) * (size_t)cap);
    for (int64_t pp = 0; pp < P0 && pp <= pos; ++pp) att[na++] = pp;
    for (int64_t j = 0; j < n_cand; ++j)
        if (sel[j])
            for (int64_t r = 0; r < C; ++r)
                if (raster_of_pos[P0 + j * C + r] >= 0) att[na++] = P0 + j * C + r;
    if (pos >= P0 && pos < vid_end) {
        for (int64_t pp = P0 + ((pos - P0) / C) * C; pp <= pos; ++pp)
            if (raster_of_pos[pp] >= 0) att[na++] = pp;
    } else if (pos >= vid_end) {
        for (int64_t pp = vid_end; pp <= pos; ++pp) att[na++] = pp;
    }
    double *w = (double *)malloc(sizeof(double) * (size_t)na);
    double mx = -INFINITY;
    for (int64_t a = 0; a < na; ++a) {
        const float *k = K + ((b * S + raster_of_pos[att[a]]) * s->Hkv + g) * D;
        double acc = 0.0;
        for (int64_t d = 0; d < D; ++d) acc += (double)q[d] * (double)k[d];
        w[a] = acc * s->scale;
        if (w[a] > mx) mx = w[a];
    }
    double Z = 0.0;
    for (int64_t a = 0; a < na; ++a) { w[a] = exp(w[a] - mx); Z += w[a]; }
    for (int64_t d = 0; d < D; ++d) out[d] = 0.0;
    for (int64_t a = 0; a < na; ++a) {
        const float *v = V + ((b * S + raster_of_pos[att[a]]) * s->Hkv + g) * D;
        double wa = w[a] / Z;
        for (int64_t d = 0; d < D; ++d) out[d] += wa * (double)v[d];
    }
    free(w);
    free(att);
    return na;
}

/* candidate cubes of the row at `pos`: none for a prefix token, the preceding cubes for a video
 * token, every cube for a text token */
static int64_t candidates_of(const adas_shape *s, int64_t pos) {
    int64_t N = n_cubes(s), C = cube_tokens(s);
    if (pos < s->n_prefix) return 0;
    if (pos < s->n_prefix + N * C) return (pos - s->n_prefix) / C;
    return N;
}

/* Evaluate a list of rows.  rows[3*i + {0,1,2}] = (batch b, query head h, raster token n).
 *   kbar        [B,Hkv,N,D] from adas_oracle_mean_keys
 *   out         (nullable) [nrows, D] fp64 attention output; NULL = selection only
 *   sel         [nrows, N] 0/1 flags (zero beyond the row's candidates)
 *   count       [nrows] |S_i|
 *   margin      (nullable) [nrows] tie margin (see adas_oracle_select_row)
 *   n_attended  (nullable) [nrows] |A|, the number of key tokens the row attends
 * Rows are independent; OpenMP splits them over the host cores. */
void adas_oracle_rows(const adas_shape *s, const float *Q, const float *K, const float *V,
                      const double *kbar, int64_t nrows, const int64_t *rows, double *out,
                      uint8_t *sel, int32_t *count, double *margin, int64_t *n_attended) {
    int64_t S = seq_len(s), N = n_cubes(s), D = s->D;
    int64_t *pos_of_raster = (int64_t *)malloc(sizeof(int64_t) * (size_t)S);
    int64_t *raster_of_pos = (int64_t *)malloc(sizeof(int64_t) * (size_t)n_positions(s));
    adas_oracle_positions(s, pos_of_raster, raster_of_pos);
    int64_t G = s->Hq / s->Hkv;
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t i = 0; i < nrows; ++i) {
        int64_t b = rows[3 * i], h = rows[3 * i + 1], n = rows[3 * i + 2];
        int64_t pos = pos_of_raster[n];
        int64_t n_cand = candidates_of(s, pos);
        const float *q = Q + ((b * S + n) * s->Hq + h) * D;
        const double *kbar_g = kbar + ((b * s->Hkv + h / G) * N) * D;
        uint8_t *sel_i = sel + i * N;
        memset(sel_i, 0, (size_t)N);
        int64_t cnt = adas_oracle_select_row(q, kbar_g, n_cand, D, s->scale, s->top_p, s->top_k, sel_i,
                                             NULL, margin ? margin + i : NULL);
        count[i] = (int32_t)cnt;
        int64_t na = -1;
        if (out) na = attend_row(s, Q, K, V, raster_of_pos, b, h, n, pos, sel_i, n_cand, out + i * D);
        if (n_attended) {
            if (na < 0) {       /* selection only: count the attended tokens without attending */
                int64_t P0 = s->n_prefix, C = cube_tokens(s), vid_end = P0 + N * C;
                na = pos < P0 ? pos + 1 : P0;
                for (int64_t j = 0; j < n_cand; ++j)
                    if (sel_i[j])
                        for (int64_t r = 0; r < C; ++r) na += raster_of_pos[P0 + j * C + r] >= 0;
                if (pos >= P0 && pos < vid_end) {
                    for (int64_t pp = P0 + ((pos - P0) / C) * C; pp <= pos; ++pp) na += raster_of_pos[pp] >= 0;
                } else if (pos >= vid_end) {
                    na += pos - vid_end + 1;
                }
            }
            n_attended[i] = na;
        }
    }
    free(pos_of_raster);
    free(raster_of_pos);
}

/* Same as adas_oracle_rows' attention step but with the selection supplied by the caller
 * (used by tests that plant a selection, e.g. "all cubes" for the dense identity). */
void adas_oracle_attend_given(const adas_shape *s, const float *Q, const float *K, const float *V,
                              int64_t nrows, const int64_t *rows, const uint8_t *sel, double *out) {
    int64_t S = seq_len(s), N = n_cubes(s), D = s->D;
    int64_t *pos_of_raster = (int64_t *)malloc(sizeof(int64_t) * (size_t)S);
    int64_t *raster_of_pos = (int64_t *)malloc(sizeof(int64_t) * (size_t)n_positions(s));
    adas_oracle_positions(s, pos_of_raster, raster_of_pos);
#pragma omp parallel for schedule(dynamic, 16)
    for (int64_t i = 0; i < nrows; ++i) {
        int64_t b = rows[3 * i], h = rows[3 * i + 1], n = rows[3 * i + 2];
        int64_t pos = pos_of_raster[n];
        attend_row(s, Q, K, V, raster_of_pos, b, h, n, pos, sel + i * N, candidates_of(s, pos), out + i * D);
    }
    free(pos_of_raster);
    free(raster_of_pos);
}
