/*
 * CPU fp64 oracle for sink+window attention over a rolling KV cache.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA
 * library is checked against.  It shares no code, header, table or constant
 * with the CUDA path, and nothing in the product may call it.
 *
 * What it follows (paper sections):
 *   - Frame sink, Sec. 3.3 "Frame Sink": the first frame chunk's tokens stay in
 *     the cache for ever and are concatenated to every attention block's K/V;
 *     the rest of the cache is a short rolling window, evicted normally.
 *   - Short-window attention, Sec. 3.3: attention restricted to a fixed
 *     temporal window of W latent frames.
 *   - KV-recache, Sec. 3.1 and Sec. 3.3 (last paragraph): at a prompt switch the
 *     cache is rebuilt from the most recent W generated frames only.
 *   - Algorithm 2 (interactive inference): every denoising pass of a chunk
 *     attends over the cache; the final clean pass commits the chunk's K/V.
 *   - Sec. 3.3 "Consistency between Training and Inference": a supervised clip
 *     of T frames is processed in one step over a resident cache of the S sink
 *     frames, the last W_a frames of the preceding context and the clip's own
 *     T frames, under the same sink + local-window rule (llo_clip; forward
 *     only, gradients are not this library's business).
 *   - Sec. 3.1: cross-attention layers alternate with the self-attention layers
 *     and inject the prompt; the recache re-encodes the prefix under the new
 *     prompt through them.  Cross-attention is plain softmax attention of the
 *     video tokens over the prompt tokens, no mask, no RoPE (llo_dense_attn).
 *
 * Readings where the paper is silent (the benchmark definition fixes them):
 *   - W counts the current chunk ("9 local + 3 sink = effective window 12").
 *   - Attention is bidirectional inside a chunk and causal across chunks.
 *   - The sink is S whole frames, S a multiple of the chunk size; recache never
 *     touches it.
 *   - 3-D RoPE (the paper does not define one): the D/2 rotation pairs are
 *     split t|h|w with n_h = n_w = floor(D/6) pairs and n_t = D/2 - 2*n_h pairs;
 *     pair j holds elements (2j, 2j+1); pair i of an axis with n_a pairs turns by
 *     pos_axis * theta^(-i/n_a).  Positions are absolute (t = frame index since
 *     the stream began).  K is cached after the rotation.
 *   - Softmax scale 1/sqrt(D).  The paper does not define the q/k normalisation of
 *     its base model; where a caller wants it fused into the append it is the RMS
 *     norm over the token's whole row of H*D elements with a learned gain
 *     (llo_rms_norm), applied before the rotation.
 *
 *   - 8-bit cache storage (the paper's appendix "Quantization" only motivates a
 *     low-precision variant; the format is this library's): rotated K and V are
 *     kept as E4M3 codes times one scale per (layer, head), see llo_set_kv_e4m3.
 *
 * Storage here is [layer][slot][token][head][dim] in double.  The slot rule
 * (frame f -> slot f if f < S, else S + (f - S) mod W) is the bit-exact
 * contract for the cache state.
 *
 * Every function states which step it is.  No blocking, fusion or reordering
 * beyond the definition; OpenMP only parallelises over independent query rows.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define LLO_OK 0
#define LLO_ERR_ARG (-1)
#define LLO_ERR_POSITION (-2)
#define LLO_ERR_NOT_RESIDENT (-3)

typedef struct llo {
    int L, H, D, P, C, S, W;
    int faithful;          /* 1: round roped Q/K to bf16 like the stored cache does */
    int64_t *end;          /* [L] frames appended so far */
    int32_t *slot_frame;   /* [L][S+W] absolute frame in each slot, -1 = empty */
    int64_t *evictions;    /* [L] frames overwritten by a newer frame */
    double *K, *V;         /* [L][S+W][P][H][D] */
    int kv_e4m3;           /* 1: rows are stored as scale * E4M3(x / scale) */
    float *k_scale, *v_scale;   /* [L][H], fp32 as the storage format defines them */
} llo;

/* ---- helpers that are not part of the method ---------------------------- */

static size_t slots(const llo *o) { return (size_t)(o->S + o->W); }
static size_t row_elems(const llo *o) { return (size_t)o->H * o->D; }
static size_t layer_elems(const llo *o) { return slots(o) * o->P * row_elems(o); }

/* Round a double to the nearest bfloat16 value (8 significant bits, ties to
 * even) and return it as a double.  Used only in storage-faithful mode. */
double llo_round_bf16(double x)
{
    if (x == 0.0 || !isfinite(x)) return x;
    int e;
    double m = frexp(x, &e);              /* x = m * 2^e, 0.5 <= |m| < 1 */
    double q = nearbyint(m * 256.0);      /* default rounding mode: ties to even */
    return ldexp(q, e - 8);
}

/* ---- 8-bit storage format -------------------------------------------------- */

/* Nearest value of the 8-bit float format E4M3: 1 sign bit, 4 exponent bits with
 * bias 7, 3 mantissa bits; no infinities; the largest finite magnitude is 448
 * (exponent field 15, mantissa 110); below 2^-6 the values are subnormal with
 * spacing 2^-9.  Ties go to the even mantissa; magnitudes beyond 448 clamp to
 * 448 (saturating conversion); NaN stays NaN. */
double llo_round_e4m3(double x)
{
    if (isnan(x) || x == 0.0) return x;
    double a = fabs(x), sgn = x < 0 ? -1.0 : 1.0;
    if (a >= 448.0) return sgn * 448.0;
    int e;
    frexp(a, &e);                         /* a = m * 2^e, 0.5 <= m < 1: binade [2^(e-1), 2^e) */
    int lsb = e - 1 - 3;                  /* exponent of the last of 3 mantissa bits in that binade */
    if (lsb < -9) lsb = -9;               /* subnormal range: fixed spacing 2^-9 */
    double q = nearbyint(ldexp(a, -lsb)); /* ties to even */
    double r = ldexp(q, lsb);
    if (r > 448.0) r = 448.0;
    return sgn * r;
}

/* The stored value of x under scale s: the division is done in fp32 (the format's
 * definition: code = E4M3(fl32(fl32(x) / s))), the product back is exact in double. */
static double store_e4m3(double x, float s)
{
    float t = (float)x / s;
    return llo_round_e4m3((double)t) * (double)s;
}

/* Switch the cache to 8-bit storage: from now on every row written by append,
 * recache or clip holds, per head h of layer l, k_scale[l*H+h] * E4M3(K / k_scale)
 * for the rotated keys and v_scale[l*H+h] * E4M3(V / v_scale) for the values.
 * Scales are positive fp32 numbers.  Rows already stored are not touched. */
int llo_set_kv_e4m3(llo *o, const float *k_scale, const float *v_scale)
{
    if (!o || !k_scale || !v_scale) return LLO_ERR_ARG;
    size_t n = (size_t)o->L * o->H;
    for (size_t i = 0; i < n; ++i)
        if (!(k_scale[i] > 0.f) || !(v_scale[i] > 0.f)) return LLO_ERR_ARG;
    if (!o->k_scale) o->k_scale = (float *)malloc(n * sizeof(float));
    if (!o->v_scale) o->v_scale = (float *)malloc(n * sizeof(float));
    if (!o->k_scale || !o->v_scale) return LLO_ERR_ARG;
    memcpy(o->k_scale, k_scale, n * sizeof(float));
    memcpy(o->v_scale, v_scale, n * sizeof(float));
    o->kv_e4m3 = 1;
    return LLO_OK;
}

/* One token's K (already rotated, in place at K) and V rows under the storage format. */
static void store_format(const llo *o, int layer, double *K, double *V)
{
    if (!o->kv_e4m3) return;
    for (int h = 0; h < o->H; ++h) {
        float ks = o->k_scale[(size_t)layer * o->H + h], vs = o->v_scale[(size_t)layer * o->H + h];
        for (int d = 0; d < o->D; ++d) {
            K[(size_t)h * o->D + d] = store_e4m3(K[(size_t)h * o->D + d], ks);
            V[(size_t)h * o->D + d] = store_e4m3(V[(size_t)h * o->D + d], vs);
        }
    }
}

/* ---- lifetime ------------------------------------------------------------ */

llo *llo_create(int L, int H, int D, int P, int C, int S, int W, int faithful)
{
    if (L <= 0 || H <= 0 || D <= 0 || (D & 1) || P <= 0 || C <= 0 || S < 0 || W <= 0)
        return NULL;
    llo *o = (llo *)calloc(1, sizeof(llo));
    if (!o) return NULL;
    o->L = L; o->H = H; o->D = D; o->P = P; o->C = C; o->S = S; o->W = W;
    o->faithful = faithful;
    o->end = (int64_t *)calloc((size_t)L, sizeof(int64_t));
    o->evictions = (int64_t *)calloc((size_t)L, sizeof(int64_t));
    o->slot_frame = (int32_t *)malloc((size_t)L * slots(o) * sizeof(int32_t));
    o->K = (double *)calloc((size_t)L * layer_elems(o), sizeof(double));
    o->V = (double *)calloc((size_t)L * layer_elems(o), sizeof(double));
    if (!o->end || !o->evictions || !o->slot_frame || !o->K || !o->V) return NULL;
    for (size_t i = 0; i < (size_t)L * slots(o); ++i) o->slot_frame[i] = -1;
    return o;
}

void llo_destroy(llo *o)
{
    if (!o) return;
    free(o->end); free(o->evictions); free(o->slot_frame); free(o->K); free(o->V);
    free(o->k_scale); free(o->v_scale);
    free(o);
}

/* Reset (Algorithm 2, "initialise KV cache C <- []"): every layer forgets
 * everything; stored bytes need not be cleared.  The eviction count is a
 * lifetime diagnostic and keeps running. */
int llo_reset(llo *o)
{
    if (!o) return LLO_ERR_ARG;
    for (int l = 0; l < o->L; ++l) o->end[l] = 0;
    for (size_t i = 0; i < (size_t)o->L * slots(o); ++i) o->slot_frame[i] = -1;
    return LLO_OK;
}

/* Skip ahead: continue the stream at frame `end` (a multiple of C, not before
 * the current end) as if the frames in between had been generated and had
 * rolled out of the window again.  The sink stays; the ring is left empty.
 * Lets a test reach a late point of a long stream by replaying only the chunks
 * that are still resident there. */
int llo_seek(llo *o, int layer, int64_t end)
{
    if (!o || layer < 0 || layer >= o->L) return LLO_ERR_ARG;
    if (end % o->C || end < o->end[layer] || end < o->S) return LLO_ERR_POSITION;
    int32_t *sf = o->slot_frame + (size_t)layer * slots(o);
    for (int s = o->S; s < o->S + o->W; ++s) sf[s] = -1;
    o->end[layer] = end;
    return LLO_OK;
}

int llo_get_state(const llo *o, int layer, int64_t *end, int32_t *slot_frame,
                  int64_t *evictions)
{
    if (!o || layer < 0 || layer >= o->L) return LLO_ERR_ARG;
    *end = o->end[layer];
    if (evictions) *evictions = o->evictions[layer];
    memcpy(slot_frame, o->slot_frame + (size_t)layer * slots(o), slots(o) * sizeof(int32_t));
    return LLO_OK;
}

/* ---- step: slot rule ------------------------------------------------------ */

/* Sink frames keep slot f for ever; later frames roll through W ring slots. */
int llo_slot_of(const llo *o, int64_t f)
{
    if (f < o->S) return (int)f;
    return o->S + (int)((f - o->S) % o->W);
}

/* ---- step: 3-D RoPE ------------------------------------------------------- */

void llo_rope_split(int D, int *n_t, int *n_h, int *n_w)
{
    *n_h = D / 6;
    *n_w = D / 6;
    *n_t = D / 2 - 2 * (D / 6);
}

/* Rotate one head row of D values sitting at grid position (t, y, x). */
static void rope_row(const double *in, double *out, int D, double theta,
                     int64_t t, int y, int x, int round_bf16)
{
    int n_t, n_h, n_w;
    llo_rope_split(D, &n_t, &n_h, &n_w);
    for (int j = 0; j < D / 2; ++j) {
        double pos; int i, n_a;
        if (j < n_t)            { pos = (double)t; i = j;             n_a = n_t; }
        else if (j < n_t + n_h) { pos = (double)y; i = j - n_t;       n_a = n_h; }
        else                    { pos = (double)x; i = j - n_t - n_h; n_a = n_w; }
        double ang = pos * pow(theta, -(double)i / (double)n_a);
        double c = cos(ang), s = sin(ang);
        double a = in[2 * j], b = in[2 * j + 1];
        double r0 = a * c - b * s;
        double r1 = a * s + b * c;
        out[2 * j]     = round_bf16 ? llo_round_bf16(r0) : r0;
        out[2 * j + 1] = round_bf16 ? llo_round_bf16(r1) : r1;
    }
}

/* RoPE over a token-major tensor [n_frames*gh*gw, H, D]; token n of a frame is
 * (y, x) = (n / gw, n % gw); frame index = frame_start + token / (gh*gw). */
int llo_rope(const double *in, double *out, int64_t n_tokens, int H, int D,
             int64_t frame_start, int gh, int gw, double theta, int round_bf16)
{
    if (!in || !out || gh <= 0 || gw <= 0 || (D & 1)) return LLO_ERR_ARG;
    int64_t P = (int64_t)gh * gw;
    for (int64_t n = 0; n < n_tokens; ++n) {
        int64_t t = frame_start + n / P;
        int y = (int)((n % P) / gw), x = (int)((n % P) % gw);
        for (int h = 0; h < H; ++h) {
            size_t off = ((size_t)n * H + h) * D;
            rope_row(in + off, out + off, D, theta, t, y, x, round_bf16);
        }
    }
    return LLO_OK;
}

/* ---- step: append (Algorithm 2, cache write; Sec. 3.3 rolling window) ----- */

/* Accepts frame_start == end (a new chunk: may evict, end += C) or
 * frame_start == end - C (overwrite the newest chunk: state unchanged). */
int llo_append(llo *o, int layer, const double *k, const double *v,
               int64_t frame_start, int n_frames, int gh, int gw, double theta)
{
    if (!o || layer < 0 || layer >= o->L || !k || !v) return LLO_ERR_ARG;
    if (n_frames != o->C || gh * gw != o->P) return LLO_ERR_ARG;
    int64_t end = o->end[layer];
    int is_new = (frame_start == end);
    int is_over = (end >= o->C && frame_start == end - o->C);
    if (!is_new && !is_over) return LLO_ERR_POSITION;

    int32_t *sf = o->slot_frame + (size_t)layer * slots(o);
    double *K = o->K + (size_t)layer * layer_elems(o);
    double *V = o->V + (size_t)layer * layer_elems(o);
    size_t re = row_elems(o);
    for (int i = 0; i < n_frames; ++i) {
        int64_t f = frame_start + i;
        int slot = llo_slot_of(o, f);
        if (sf[slot] >= 0 && sf[slot] != f) o->evictions[layer] += 1;
        sf[slot] = (int32_t)f;
        for (int n = 0; n < o->P; ++n) {
            int y = n / gw, x = n % gw;
            size_t src = ((size_t)i * o->P + n) * re;
            size_t dst = ((size_t)slot * o->P + n) * re;
            for (int h = 0; h < o->H; ++h)
                rope_row(k + src + (size_t)h * o->D, K + dst + (size_t)h * o->D,
                         o->D, theta, f, y, x, o->faithful);
            memcpy(V + dst, v + src, re * sizeof(double));
            store_format(o, layer, K + dst, V + dst);
        }
    }
    if (is_new) o->end[layer] = end + o->C;
    return LLO_OK;
}

/* ---- step: visible set ---------------------------------------------------- */

/* Frame fk is visible to a query in frame fq iff it is not in a later chunk
 * and it is either a sink frame or inside the W-frame window that ends with the
 * query's chunk.  lo_floor additionally hides non-sink frames older than it
 * (recache: frames that no longer exist). */
static int visible_in_window(const llo *o, int64_t fq, int64_t fk, int64_t lo_floor, int window)
{
    int64_t hi = (fq / o->C + 1) * o->C;      /* one past the query's chunk */
    if (fk < 0 || fk >= hi) return 0;
    if (fk < o->S) return 1;
    return fk >= hi - window && fk >= lo_floor;
}

int llo_visible(const llo *o, int64_t fq, int64_t fk, int64_t lo_floor)
{
    return visible_in_window(o, fq, fk, lo_floor, o->W);
}

/* The same with a local window of `window` frames that may be shorter than the
 * resident ring (the clip step below). */
int llo_visible_window(const llo *o, int64_t fq, int64_t fk, int window)
{
    return visible_in_window(o, fq, fk, 0, window);
}

/* ---- step: attention ------------------------------------------------------ */

/* Softmax attention of selected query rows over their visible keys.
 *   q_roped [n_q_frames*P, H, D] : queries after RoPE
 *   rows[n_rows]                 : query row indices to evaluate (NULL = all)
 *   out [n_rows, H, D], lse [n_rows, H] (natural log of the softmax denominator)
 * Per row and head: s_j = q.k_j / sqrt(D), p = softmax(s), o = sum p_j v_j. */
static int attn_in_window(const llo *o, int layer, const double *q_roped, int64_t q_frame_start,
                          int n_q_frames, int64_t lo_floor, int window, const int64_t *rows, int64_t n_rows,
                          double *out, double *lse)
{
    if (!o || layer < 0 || layer >= o->L || !q_roped || !out) return LLO_ERR_ARG;
    int64_t nq = (int64_t)n_q_frames * o->P;
    if (!rows) n_rows = nq;
    const int32_t *sf = o->slot_frame + (size_t)layer * slots(o);
    const double *K = o->K + (size_t)layer * layer_elems(o);
    const double *V = o->V + (size_t)layer * layer_elems(o);
    const int H = o->H, D = o->D, P = o->P;
    const double scale = 1.0 / sqrt((double)D);
    int status = LLO_OK;

#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t ri = 0; ri < n_rows; ++ri) {
        int64_t r = rows ? rows[ri] : ri;
        if (r < 0 || r >= nq) { status = LLO_ERR_ARG; continue; }
        int64_t fq = q_frame_start + r / P;
        int64_t hi = (fq / o->C + 1) * o->C;
        /* visible frames -> slots; every visible frame must be resident */
        int nvis = 0;
        int *vslot = (int *)malloc(sizeof(int) * (size_t)(o->S + o->W));
        for (int64_t fk = 0; fk < hi; ++fk) {
            if (!visible_in_window(o, fq, fk, lo_floor, window)) continue;
            int slot = llo_slot_of(o, fk);
            if (sf[slot] != (int32_t)fk || nvis >= o->S + o->W) { status = LLO_ERR_NOT_RESIDENT; nvis = -1; break; }
            vslot[nvis++] = slot;
        }
        if (nvis <= 0) { free(vslot); if (nvis == 0) status = LLO_ERR_NOT_RESIDENT; continue; }
        int64_t nk = (int64_t)nvis * P;
        double *s = (double *)malloc(sizeof(double) * (size_t)nk);
        for (int h = 0; h < H; ++h) {
            const double *qv = q_roped + ((size_t)r * H + h) * D;
            double m = -INFINITY;
            for (int a = 0; a < nvis; ++a)
                for (int n = 0; n < P; ++n) {
                    const double *kv = K + (((size_t)vslot[a] * P + n) * H + h) * D;
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d) dot += qv[d] * kv[d];
                    dot *= scale;
                    s[(size_t)a * P + n] = dot;
                    if (dot > m) m = dot;
                }
            double denom = 0.0;
            for (int64_t j = 0; j < nk; ++j) { s[j] = exp(s[j] - m); denom += s[j]; }
            double *ov = out + ((size_t)ri * H + h) * D;
            for (int d = 0; d < D; ++d) ov[d] = 0.0;
            for (int a = 0; a < nvis; ++a)
                for (int n = 0; n < P; ++n) {
                    double p = s[(size_t)a * P + n] / denom;
                    const double *vv = V + (((size_t)vslot[a] * P + n) * H + h) * D;
                    for (int d = 0; d < D; ++d) ov[d] += p * vv[d];
                }
            if (lse) lse[(size_t)ri * H + h] = m + log(denom);
        }
        free(s); free(vslot);
    }
    return status;
}

int llo_attn(const llo *o, int layer, const double *q_roped, int64_t q_frame_start,
             int n_q_frames, int64_t lo_floor, const int64_t *rows, int64_t n_rows,
             double *out, double *lse)
{
    if (!o) return LLO_ERR_ARG;
    return attn_in_window(o, layer, q_roped, q_frame_start, n_q_frames, lo_floor, o->W, rows, n_rows, out, lse);
}

/* Softmax probabilities of one (row, head) and the cache rows they belong to;
 * for tiny cases (checks that rows sum to one, and which keys are seen).
 * key_rows[j] = slot*P + token.  Returns the number of visible keys or <0. */
int64_t llo_attn_probs(const llo *o, int layer, const double *q_roped, int64_t q_frame_start,
                       int64_t lo_floor, int64_t row, int head, double *probs,
                       int64_t *key_rows, int64_t cap)
{
    if (!o || layer < 0 || layer >= o->L) return LLO_ERR_ARG;
    const int32_t *sf = o->slot_frame + (size_t)layer * slots(o);
    const double *K = o->K + (size_t)layer * layer_elems(o);
    const int H = o->H, D = o->D, P = o->P;
    int64_t fq = q_frame_start + row / P;
    int64_t hi = (fq / o->C + 1) * o->C;
    int64_t nk = 0;
    const double *qv = q_roped + ((size_t)row * H + head) * D;
    double m = -INFINITY;
    for (int64_t fk = 0; fk < hi; ++fk) {
        if (!llo_visible(o, fq, fk, lo_floor)) continue;
        int slot = llo_slot_of(o, fk);
        if (sf[slot] != (int32_t)fk) return LLO_ERR_NOT_RESIDENT;
        for (int n = 0; n < P; ++n) {
            if (nk >= cap) return LLO_ERR_ARG;
            const double *kv = K + (((size_t)slot * P + n) * H + head) * D;
            double dot = 0.0;
            for (int d = 0; d < D; ++d) dot += qv[d] * kv[d];
            probs[nk] = dot / sqrt((double)D);
            key_rows[nk] = (int64_t)slot * P + n;
            if (probs[nk] > m) m = probs[nk];
            ++nk;
        }
    }
    double denom = 0.0;
    for (int64_t j = 0; j < nk; ++j) { probs[j] = exp(probs[j] - m); denom += probs[j]; }
    for (int64_t j = 0; j < nk; ++j) probs[j] /= denom;
    return nk;
}

/* ---- step: recache (Sec. 3.1; Sec. 3.3 last paragraph) --------------------- */

/* Rebuild the ring from fresh K/V of the resident window frames
 * [r0, end), r0 = max(S, end - W): re-rope and overwrite their rows (slot table,
 * end and sink untouched), then attend all those frames' queries under the
 * block-causal visible set.  q_roped_out (nullable) receives the roped queries.
 * n_frames must equal end - r0 (0 when only sink frames exist: no work). */
int llo_recache(llo *o, int layer, const double *q, const double *k, const double *v,
                int n_frames, int gh, int gw, double theta,
                const int64_t *rows, int64_t n_rows,
                double *q_roped_out, double *out, double *lse)
{
    if (!o || layer < 0 || layer >= o->L) return LLO_ERR_ARG;
    if (gh * gw != o->P) return LLO_ERR_ARG;
    int64_t end = o->end[layer];
    int64_t r0 = end - o->W; if (r0 < o->S) r0 = o->S;
    int64_t resident = end - r0; if (resident < 0) resident = 0;
    if (n_frames != resident) return LLO_ERR_POSITION;
    if (n_frames == 0) return LLO_OK;
    if (!q || !k || !v || !out) return LLO_ERR_ARG;

    const int32_t *sf = o->slot_frame + (size_t)layer * slots(o);
    double *K = o->K + (size_t)layer * layer_elems(o);
    double *V = o->V + (size_t)layer * layer_elems(o);
    size_t re = row_elems(o);
    for (int i = 0; i < n_frames; ++i) {
        int64_t f = r0 + i;
        int slot = llo_slot_of(o, f);
        if (sf[slot] != (int32_t)f) return LLO_ERR_NOT_RESIDENT;
        for (int n = 0; n < o->P; ++n) {
            int y = n / gw, x = n % gw;
            size_t src = ((size_t)i * o->P + n) * re;
            size_t dst = ((size_t)slot * o->P + n) * re;
            for (int h = 0; h < o->H; ++h)
                rope_row(k + src + (size_t)h * o->D, K + dst + (size_t)h * o->D,
                         o->D, theta, f, y, x, o->faithful);
            memcpy(V + dst, v + src, re * sizeof(double));
            store_format(o, layer, K + dst, V + dst);
        }
    }
    int64_t nq = (int64_t)n_frames * o->P;
    double *qr = q_roped_out ? q_roped_out : (double *)malloc(sizeof(double) * (size_t)nq * re);
    llo_rope(q, qr, nq, o->H, o->D, r0, gh, gw, theta, o->faithful);
    int st = llo_attn(o, layer, qr, r0, n_frames, r0, rows, n_rows, out, lse);
    if (!q_roped_out) free(qr);
    return st;
}

/* ---- step: a clip in one go (Sec. 3.3, "Consistency between Training and Inference") ---- */

/* The clip's n_frames frames (whole chunks, starting at the stream's end) enter
 * the cache chunk after chunk exactly as in llo_append; then every clip frame's
 * queries attend over the sink frames and the local window of `window` frames
 * that ends with their own chunk: the tail of the preceding context and the
 * clip's earlier chunks.  The ring must be long enough that the first chunk's
 * window is still resident once the last chunk is in:
 * W >= window + n_frames - C.  q_roped_out (nullable) receives the roped queries. */
int llo_clip(llo *o, int layer, const double *q, const double *k, const double *v,
             int64_t frame_start, int n_frames, int window, int gh, int gw, double theta,
             const int64_t *rows, int64_t n_rows, double *q_roped_out, double *out, double *lse)
{
    if (!o || layer < 0 || layer >= o->L || !q || !k || !v || !out) return LLO_ERR_ARG;
    if (gh * gw != o->P || n_frames <= 0 || n_frames % o->C) return LLO_ERR_ARG;
    if (window < o->C || window % o->C || window + n_frames - o->C > o->W) return LLO_ERR_ARG;
    if (frame_start != o->end[layer]) return LLO_ERR_POSITION;
    size_t chunk_elems = (size_t)o->C * o->P * row_elems(o);
    for (int c = 0; c < n_frames / o->C; ++c) {
        int st = llo_append(o, layer, k + (size_t)c * chunk_elems, v + (size_t)c * chunk_elems,
                            frame_start + (int64_t)c * o->C, o->C, gh, gw, theta);
        if (st != LLO_OK) return st;
    }
    int64_t nq = (int64_t)n_frames * o->P;
    double *qr = q_roped_out ? q_roped_out : (double *)malloc(sizeof(double) * (size_t)nq * row_elems(o));
    llo_rope(q, qr, nq, o->H, o->D, frame_start, gh, gw, theta, o->faithful);
    int st = attn_in_window(o, layer, qr, frame_start, n_frames, 0, window, rows, n_rows, out, lse);
    if (!q_roped_out) free(qr);
    return st;
}

/* ---- step: gradients of the clip step (Sec. 3.3, "Consistency between Training and Inference":
 * the clip's T frames carry gradients, the sink and the preceding context are detached;
 * Algorithm 1 back-propagates the loss of the newest clip only) ------------------------------- */

/* The inverse of rope_row: rotate every pair by minus its angle (the rotation is orthogonal,
 * so the gradient with respect to the unrotated row is the rotated gradient turned back). */
static void rope_row_back(const double *in, double *out, int D, double theta, int64_t t, int y, int x)
{
    int n_t, n_h, n_w;
    llo_rope_split(D, &n_t, &n_h, &n_w);
    for (int j = 0; j < D / 2; ++j) {
        double pos; int i, n_a;
        if (j < n_t)            { pos = (double)t; i = j;             n_a = n_t; }
        else if (j < n_t + n_h) { pos = (double)y; i = j - n_t;       n_a = n_h; }
        else                    { pos = (double)x; i = j - n_t - n_h; n_a = n_w; }
        double ang = pos * pow(theta, -(double)i / (double)n_a);
        double c = cos(ang), s = sin(ang);
        double a = in[2 * j], b = in[2 * j + 1];
        out[2 * j]     = a * c + b * s;
        out[2 * j + 1] = -a * s + b * c;
    }
}

/* Given the cache as llo_clip left it, the clip's unrotated queries q and the gradient d_out of
 * a scalar loss with respect to the clip's attention output, the gradients with respect to the
 * clip's q, k and v as they were handed to llo_clip (before the rotation), all [n_frames*P, H, D].
 * With s_ij = q_i.k_j / sqrt(D) over the keys j visible to row i, p = softmax(s), o_i = sum p_ij v_j:
 *   delta_i = d_out_i . o_i,  dP_ij = d_out_i . v_j,  dS_ij = p_ij (dP_ij - delta_i),
 *   dq_i = sum_j dS_ij k_j / sqrt(D),  dk_j = sum_i dS_ij q_i / sqrt(D),  dv_j = sum_i p_ij d_out_i,
 * (q, k after rotation), dk and dv only for keys that are frames of the clip, then dq and dk
 * turned back through the rotation.  mag_* (nullable, same shapes) receive the sums of the
 * absolute values of the terms each gradient element adds up (dq, dk: in the rotated frame,
 * summed over the element's rotation pair): the scale of its rounding error. */
int llo_clip_backward(const llo *o, int layer, const double *q, const double *d_out,
                      int64_t frame_start, int n_frames, int window, int gh, int gw, double theta,
                      double *dq, double *dk, double *dv, double *mag_q, double *mag_k, double *mag_v)
{
    if (!o || layer < 0 || layer >= o->L || !q || !d_out || !dq || !dk || !dv) return LLO_ERR_ARG;
    if (gh * gw != o->P || n_frames <= 0 || n_frames % o->C) return LLO_ERR_ARG;
    if (frame_start + n_frames != o->end[layer]) return LLO_ERR_POSITION;
    const int H = o->H, D = o->D, P = o->P;
    const int64_t nq = (int64_t)n_frames * P;
    const size_t re = row_elems(o);
    const double scale = 1.0 / sqrt((double)D);
    const int32_t *sf = o->slot_frame + (size_t)layer * slots(o);
    const double *K = o->K + (size_t)layer * layer_elems(o);
    const double *V = o->V + (size_t)layer * layer_elems(o);
    double *qr = (double *)malloc(sizeof(double) * (size_t)nq * re);
    double *lse = (double *)malloc(sizeof(double) * (size_t)nq * H);
    double *delta = (double *)malloc(sizeof(double) * (size_t)nq * H);
    double *dq_r = (double *)calloc((size_t)nq * re, sizeof(double));      /* gradients in the rotated frame */
    double *dk_r = (double *)calloc((size_t)nq * re, sizeof(double));
    double *mq = (double *)calloc((size_t)nq * re, sizeof(double));
    double *mk = (double *)calloc((size_t)nq * re, sizeof(double));
    if (!qr || !lse || !delta || !dq_r || !dk_r || !mq || !mk) return LLO_ERR_ARG;
    llo_rope(q, qr, nq, H, D, frame_start, gh, gw, theta, o->faithful);
    memset(dv, 0, sizeof(double) * (size_t)nq * re);
    if (mag_v) memset(mag_v, 0, sizeof(double) * (size_t)nq * re);
    int status = LLO_OK;

    /* pass 1, per query row: softmax statistics, delta, dq */
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t r = 0; r < nq; ++r) {
        int64_t fq = frame_start + r / P;
        int64_t hi = (fq / o->C + 1) * o->C;
        for (int h = 0; h < H; ++h) {
            const double *qv = qr + ((size_t)r * H + h) * D;
            const double *go = d_out + ((size_t)r * H + h) * D;
            /* scores over the visible keys */
            double m = -INFINITY, denom = 0.0;
            for (int pass = 0; pass < 2; ++pass)
                for (int64_t fk = 0; fk < hi; ++fk) {
                    if (!visible_in_window(o, fq, fk, 0, window)) continue;
                    int slot = llo_slot_of(o, fk);
                    if (sf[slot] != (int32_t)fk) { status = LLO_ERR_NOT_RESIDENT; continue; }
                    for (int n = 0; n < P; ++n) {
                        const double *kv = K + (((size_t)slot * P + n) * H + h) * D;
                        double dot = 0.0;
                        for (int d = 0; d < D; ++d) dot += qv[d] * kv[d];
                        dot *= scale;
                        if (pass == 0) { if (dot > m) m = dot; } else denom += exp(dot - m);
                    }
                }
            double l = m + log(denom);
            lse[(size_t)r * H + h] = l;
            /* o_i and delta_i */
            double dl = 0.0;
            double *ov = (double *)calloc((size_t)D, sizeof(double));
            for (int64_t fk = 0; fk < hi; ++fk) {
                if (!visible_in_window(o, fq, fk, 0, window)) continue;
                int slot = llo_slot_of(o, fk);
                for (int n = 0; n < P; ++n) {
                    const double *kv = K + (((size_t)slot * P + n) * H + h) * D;
                    const double *vv = V + (((size_t)slot * P + n) * H + h) * D;
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d) dot += qv[d] * kv[d];
                    double p = exp(dot * scale - l);
                    for (int d = 0; d < D; ++d) ov[d] += p * vv[d];
                }
            }
            for (int d = 0; d < D; ++d) dl += go[d] * ov[d];
            free(ov);
            delta[(size_t)r * H + h] = dl;
            /* dq_i */
            double *gq = dq_r + ((size_t)r * H + h) * D, *gm = mq + ((size_t)r * H + h) * D;
            for (int64_t fk = 0; fk < hi; ++fk) {
                if (!visible_in_window(o, fq, fk, 0, window)) continue;
                int slot = llo_slot_of(o, fk);
                for (int n = 0; n < P; ++n) {
                    const double *kv = K + (((size_t)slot * P + n) * H + h) * D;
                    const double *vv = V + (((size_t)slot * P + n) * H + h) * D;
                    double dot = 0.0, dp = 0.0;
                    for (int d = 0; d < D; ++d) { dot += qv[d] * kv[d]; dp += go[d] * vv[d]; }
                    double p = exp(dot * scale - l);
                    double ds = p * (dp - dl) * scale;
                    for (int d = 0; d < D; ++d) { gq[d] += ds * kv[d]; gm[d] += fabs(ds * kv[d]); }
                }
            }
        }
    }

    /* pass 2, per key row of the clip: dk_j and dv_j over the query rows that see it */
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t j = 0; j < nq; ++j) {
        int64_t fk = frame_start + j / P;
        int slot = llo_slot_of(o, fk);
        int n = (int)(j % P);
        for (int h = 0; h < H; ++h) {
            const double *kv = K + (((size_t)slot * P + n) * H + h) * D;
            const double *vv = V + (((size_t)slot * P + n) * H + h) * D;
            double *gk = dk_r + ((size_t)j * H + h) * D, *gkm = mk + ((size_t)j * H + h) * D;
            double *gv = dv + ((size_t)j * H + h) * D;
            double *gvm = mag_v ? mag_v + ((size_t)j * H + h) * D : NULL;
            for (int64_t r = 0; r < nq; ++r) {
                int64_t fq = frame_start + r / P;
                if (!visible_in_window(o, fq, fk, 0, window)) continue;
                const double *qv = qr + ((size_t)r * H + h) * D;
                const double *go = d_out + ((size_t)r * H + h) * D;
                double dot = 0.0, dp = 0.0;
                for (int d = 0; d < D; ++d) { dot += qv[d] * kv[d]; dp += go[d] * vv[d]; }
                double p = exp(dot * scale - lse[(size_t)r * H + h]);
                double ds = p * (dp - delta[(size_t)r * H + h]) * scale;
                for (int d = 0; d < D; ++d) {
                    gk[d] += ds * qv[d]; gkm[d] += fabs(ds * qv[d]);
                    gv[d] += p * go[d];
                    if (gvm) gvm[d] += fabs(p * go[d]);
                }
            }
        }
    }

    /* back through the rotation */
    for (int64_t r = 0; r < nq; ++r) {
        int64_t t = frame_start + r / P;
        int y = (int)((r % P) / gw), x = (int)((r % P) % gw);
        for (int h = 0; h < H; ++h) {
            size_t off = ((size_t)r * H + h) * D;
            rope_row_back(dq_r + off, dq + off, D, theta, t, y, x);
            rope_row_back(dk_r + off, dk + off, D, theta, t, y, x);
            for (int d = 0; d < D; d += 2) {
                if (mag_q) mag_q[off + d] = mag_q[off + d + 1] = mq[off + d] + mq[off + d + 1];
                if (mag_k) mag_k[off + d] = mag_k[off + d + 1] = mk[off + d] + mk[off + d + 1];
            }
        }
    }
    free(qr); free(lse); free(delta); free(dq_r); free(dk_r); free(mq); free(mk);
    return status;
}

/* ---- step: RMS norm of q and k rows (upstream of the rotation) ---------------- */

/* y[t][e] = x[t][e] / sqrt(mean_e(x[t][e]^2) + eps) * gain[e], e over the token's
 * whole row of n_elems = H*D elements. */
int llo_rms_norm(const double *x, const double *gain, double eps, int64_t n_tokens, int n_elems, double *y)
{
    if (!x || !gain || !y || n_tokens < 0 || n_elems <= 0) return LLO_ERR_ARG;
    for (int64_t t = 0; t < n_tokens; ++t) {
        const double *xr = x + (size_t)t * n_elems;
        double ms = 0.0;
        for (int e = 0; e < n_elems; ++e) ms += xr[e] * xr[e];
        ms /= (double)n_elems;
        double r = 1.0 / sqrt(ms + eps);
        for (int e = 0; e < n_elems; ++e) y[(size_t)t * n_elems + e] = xr[e] * r * gain[e];
    }
    return LLO_OK;
}

/* ---- step: dense attention (cross-attention to the prompt, Sec. 3.1) -------- */

/* o = softmax(q k^T / sqrt(D)) v per head; every query sees every key.
 *   q [n_q, H, D], k and v [n_k, H, D]; rows[n_rows] selects query rows (NULL = all)
 *   out [n_rows, H, D], lse [n_rows, H] (nullable). */
int llo_dense_attn(const double *q, const double *k, const double *v, int64_t n_q, int64_t n_k,
                   int H, int D, const int64_t *rows, int64_t n_rows, double *out, double *lse)
{
    if (!q || !k || !v || !out || n_q <= 0 || n_k <= 0 || H <= 0 || D <= 0) return LLO_ERR_ARG;
    if (!rows) n_rows = n_q;
    const double scale = 1.0 / sqrt((double)D);
    int status = LLO_OK;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t ri = 0; ri < n_rows; ++ri) {
        int64_t r = rows ? rows[ri] : ri;
        if (r < 0 || r >= n_q) { status = LLO_ERR_ARG; continue; }
        double *s = (double *)malloc(sizeof(double) * (size_t)n_k);
        for (int h = 0; h < H; ++h) {
            const double *qv = q + ((size_t)r * H + h) * D;
            double m = -INFINITY;
            for (int64_t j = 0; j < n_k; ++j) {
                const double *kv = k + ((size_t)j * H + h) * D;
                double dot = 0.0;
                for (int d = 0; d < D; ++d) dot += qv[d] * kv[d];
                s[j] = dot * scale;
                if (s[j] > m) m = s[j];
            }
            double denom = 0.0;
            for (int64_t j = 0; j < n_k; ++j) { s[j] = exp(s[j] - m); denom += s[j]; }
            double *ov = out + ((size_t)ri * H + h) * D;
            for (int d = 0; d < D; ++d) ov[d] = 0.0;
            for (int64_t j = 0; j < n_k; ++j) {
                double pj = s[j] / denom;
                const double *vv = v + ((size_t)j * H + h) * D;
                for (int d = 0; d < D; ++d) ov[d] += pj * vv[d];
            }
            if (lse) lse[(size_t)ri * H + h] = m + log(denom);
        }
        free(s);
    }
    return status;
}

/* Read back one cache row (slot*P + token) of K and V, [H, D] each. */
int llo_read_row(const llo *o, int layer, int64_t cache_row, double *k_out, double *v_out)
{
    if (!o || layer < 0 || layer >= o->L) return LLO_ERR_ARG;
    if (cache_row < 0 || cache_row >= (int64_t)slots(o) * o->P) return LLO_ERR_ARG;
    size_t off = (size_t)layer * layer_elems(o) + (size_t)cache_row * row_elems(o);
    memcpy(k_out, o->K + off, row_elems(o) * sizeof(double));
    memcpy(v_out, o->V + off, row_elems(o) * sizeof(double));
    return LLO_OK;
}

/* Bulk read of a layer's cache, [S+W, P, H, D] each. */
int llo_read_layer(const llo *o, int layer, double *k_out, double *v_out)
{
    if (!o || layer < 0 || layer >= o->L) return LLO_ERR_ARG;
    size_t off = (size_t)layer * layer_elems(o);
    memcpy(k_out, o->K + off, layer_elems(o) * sizeof(double));
    memcpy(v_out, o->V + off, layer_elems(o) * sizeof(double));
    return LLO_OK;
}
