/*
 * TreeKV oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, fp64 CPU statement of TreeKV (arXiv 2501.04987): attention
 * over a fixed-size KV cache, the averaged-attention importance score, and the
 * cycling adjacent-pair eviction of Algorithm 1, written step by step in the
 * paper's order.  Only tests, the smoke check and the CPU-baseline leg of the
 * benchmark may load this library.  It shares no code with the CUDA library.
 *
 * State per unit (sequence, KV head): ordered lists K[len][d], V[len][d],
 * S[len] (sum of attention received, Alg. 1 "S") and pos[len] (0-based stream
 * index of the token in the slot).  The paper's counter C (Alg. 1 "C", number
 * of steps a token has been present) is kept explicitly as well, so that the
 * identity C_j = N_seen - pos_j is something the tests can check instead of
 * something the oracle assumes.
 * State per sequence: N_seen (tokens fed so far), idx (1-based eviction
 * pointer, Alg. 1 "idx", initial value 1), n_evicted.
 *
 * Readings of the paper used here (each is a switch or a comment below):
 *   - idx update: the prose of Section 4.1 ("Eviction Scope") says idx cycles
 *     1,2,...,c; that is idx <- (idx mod c) + 1.  The formula as printed in
 *     Algorithm 1, idx <- (idx+1) mod c + 1, is available as
 *     TKVO_IDX_LITERAL for documentation; it skips slots.
 *   - ties and NaN: Algorithm 1 tests "S_idx > S_idx+1" strictly, so anything
 *     else evicts slot idx (the older one).
 *   - sqrt(d) of Section 3.1 is sqrt(head_dim).
 *   - grouped-query attention (not in the paper): the attention weight a KV
 *     head's slot receives in a step is the mean over the query heads of its
 *     group; with one query head per KV head this is Algorithm 1 unchanged.
 *   - chunked prefill (not in the paper): m tokens are appended, row i of the
 *     chunk attends to every slot whose pos <= its own, S and C are advanced
 *     for all m steps at once, then Algorithm 1's eviction branch is repeated
 *     with those frozen scores until the length is back to c.
 *   - protected tokens (Section 5.2: a cache of 1024 split into 4 initial, 508 recent and 512 method-chosen tokens; the
 *     paper does not say how the three parts interact): the first n_sink tokens of the stream and the newest
 *     n_recent cached tokens are never in an eviction scope.  Algorithm 1 runs on the region between them, whose
 *     size is c_mid = c - n_sink - n_recent: the scope is slots {n_sink + idx, n_sink + idx + 1} of the whole
 *     cache and idx cycles 1..c_mid.  A token becomes eligible in the step in which it stops being one of the
 *     n_recent newest (it is then the last slot of the middle region, exactly where Algorithm 1 appends).  S and
 *     C of every cached token, protected or not, advance as in Algorithm 1 from the token's arrival.  With
 *     n_sink = n_recent = 0 this is Algorithm 1 unchanged.
 *   - one-shot, block-level prefill (Section 4.2): the prompt is cut into blocks of b tokens, each block
 *     standing for one token of Algorithm 1; the last block is the observation window whose b queries score the
 *     whole prompt: Algorithm 1's S and C updates are applied for those b rows only, so a token older than the
 *     window has C = b and window token u (0-based) has C = b - u; a block's score is the mean of its tokens'
 *     S/C; Algorithm 1's branch then runs on blocks with a cache of c / b blocks, blocks arriving in order.  The
 *     output is plain causal attention over the whole prompt.  Afterwards the token-level pointer is the first
 *     token of the block the block pointer stands on, idx = (idx_blocks - 1) b + 1, which equals
 *     (tokens evicted mod c) + 1.  The paper gives neither b nor the treatment of a ragged tail: the prompt
 *     length and c must be multiples of b here.  S and C carry on into decoding as they are.
 *   - in-cache positions (Section 4.1 "Position Encoding"): positional encodings are re-assigned after eviction,
 *     i.e. the token in cache slot j (0-based) is encoded at position j and the query at its own slot.  With
 *     this switched on, q and k arrive WITHOUT positional encoding, the cache keeps k as given, and attention
 *     applies rotary embedding (rotate-half pairing (t, t + d/2)) from a cos / sin table indexed by slot.  The
 *     numeric contract follows the paper's "bf16 precision" set-up: the rotated q and k are computed in fp32 as
 *     x1' = fma(x1, cos, -(x2 sin)), x2' = fma(x2, cos, x1 sin) and rounded to the cache's element type before
 *     the fp64 dot product (no rounding for an fp32 cache).
 *   - accumulated criterion (Section 4.1 "Importance Score" reports that criteria other than the average were
 *     tried, among them the accumulated weight, the only one with an evident definition): TKVO_RULE_ACCUMULATED
 *     compares S instead of S-bar = S / C in Algorithm 1's branch, and block means of S in the one-shot
 *     prefill.  Pinned by a dictionary restatement and by the closed form under uniform attention (the older
 *     token has the larger sum, so the left member always survives: the keep-left ladder).
 *   PARITY UNPINNED: the grouped-query, chunked-prefill, protected-token, one-shot and in-cache-position
 *   readings are not fixed by anything the paper prints; the tests constrain them (m=1 equals a decode step,
 *   mass conservation, score-free rules give identical retained sets) but cannot pin them to the paper.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define TKVO_RULE_SCORES 0     /* Algorithm 1 */
#define TKVO_RULE_KEEP_LEFT 1  /* Section 5.4 ablation: always keep slot idx */
#define TKVO_RULE_EVICT_LEFT 2 /* what an exact tie does: always evict slot idx */
#define TKVO_RULE_ACCUMULATED 3 /* Section 4.1 "Importance Score": the accumulated attention weight, a criterion the
                                   authors also tried: Algorithm 1 with S in place of S-bar = S / C */

#define TKVO_IDX_CYCLE 0   /* idx <- (idx mod c) + 1   (prose of Section 4.1) */
#define TKVO_IDX_LITERAL 1 /* idx <- (idx+1) mod c + 1 (Algorithm 1 as printed) */

typedef struct {
    int len, cap;
    double *K, *V; /* [cap][d] */
    double *S;     /* [cap] */
    int64_t *C;    /* [cap] */
    int64_t *pos;  /* [cap] */
} tkvo_unit;

typedef struct {
    int c, Hq, Hkv, d, B, g;
    int n_sink, n_recent; /* protected tokens at both ends (Section 5.2); 0, 0 = Algorithm 1 as printed */
    /* in-cache positions (Section 4.1 "Position Encoding"): rotary tables by slot, NULL = position-agnostic */
    const float *rope_cos, *rope_sin; /* [rope_slots][d/2], owned by the caller */
    int rope_slots, rope_round_bf16;
    /* block-level eviction pending after tkvo_prefill_oneshot_attend */
    int *pending_block; /* [B], 0 = none */
    int rule, idx_mode;
    int64_t *n_seen;    /* [B] */
    int64_t *n_evicted; /* [B] */
    int *idx;           /* [B], 1-based */
    tkvo_unit *u;       /* [B*Hkv] */
    /* diagnostics of the last tkvo_evict call */
    int64_t last_near_ties;
    int64_t last_hint_flips;
    double last_min_gap;
    /* totals */
    int64_t total_near_ties;
    int64_t total_hint_flips;
} tkvo;

static void unit_reserve(tkvo_unit *u, int d, int need) {
    if (need <= u->cap) return;
    int cap = u->cap ? u->cap : 16;
    while (cap < need) cap *= 2;
    u->K = (double *)realloc(u->K, sizeof(double) * (size_t)cap * d);
    u->V = (double *)realloc(u->V, sizeof(double) * (size_t)cap * d);
    u->S = (double *)realloc(u->S, sizeof(double) * (size_t)cap);
    u->C = (int64_t *)realloc(u->C, sizeof(int64_t) * (size_t)cap);
    u->pos = (int64_t *)realloc(u->pos, sizeof(int64_t) * (size_t)cap);
    u->cap = cap;
}

/* Algorithm 1, initialisation: empty tensors, idx = 1. */
tkvo *tkvo_create(int budget, int n_heads, int n_kv_heads, int head_dim, int batch) {
    if (budget < 2 || n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads || head_dim < 1 || batch < 1) return NULL;
    tkvo *o = (tkvo *)calloc(1, sizeof(tkvo));
    o->c = budget; o->Hq = n_heads; o->Hkv = n_kv_heads; o->d = head_dim; o->B = batch;
    o->g = n_heads / n_kv_heads;
    o->rule = TKVO_RULE_SCORES; o->idx_mode = TKVO_IDX_CYCLE;
    o->n_seen = (int64_t *)calloc((size_t)batch, sizeof(int64_t));
    o->n_evicted = (int64_t *)calloc((size_t)batch, sizeof(int64_t));
    o->idx = (int *)malloc(sizeof(int) * (size_t)batch);
    for (int b = 0; b < batch; ++b) o->idx[b] = 1;
    o->u = (tkvo_unit *)calloc((size_t)batch * n_kv_heads, sizeof(tkvo_unit));
    o->pending_block = (int *)calloc((size_t)batch, sizeof(int));
    o->last_min_gap = INFINITY;
    return o;
}

void tkvo_destroy(tkvo *o) {
    if (!o) return;
    for (int i = 0; i < o->B * o->Hkv; ++i) {
        free(o->u[i].K); free(o->u[i].V); free(o->u[i].S); free(o->u[i].C); free(o->u[i].pos);
    }
    free(o->u); free(o->n_seen); free(o->n_evicted); free(o->idx); free(o->pending_block); free(o);
}

void tkvo_set_rule(tkvo *o, int rule) { o->rule = rule; }

/* Section 5.2: keep the first n_sink tokens and the newest n_recent tokens out of every eviction scope.
 * Only valid before the first token; the middle region must keep room for a scope. Returns 0 on success. */
int tkvo_set_protection(tkvo *o, int n_sink, int n_recent) {
    if (n_sink < 0 || n_recent < 0 || o->c - n_sink - n_recent < 2) return -1;
    for (int b = 0; b < o->B; ++b) if (o->n_seen[b] != 0) return -2;
    o->n_sink = n_sink; o->n_recent = n_recent;
    return 0;
}
void tkvo_set_idx_mode(tkvo *o, int mode) { o->idx_mode = mode; }

/* Append one token to every KV head of sequence b (Alg. 1, the two append
 * steps), with S = 0 and C = 0 for the new slot (the "union {0}" of the C and S updates). */
static void append_token(tkvo *o, int b, const double *k, const double *v) {
    for (int h = 0; h < o->Hkv; ++h) {
        tkvo_unit *u = &o->u[b * o->Hkv + h];
        unit_reserve(u, o->d, u->len + 1);
        memcpy(u->K + (size_t)u->len * o->d, k + (size_t)h * o->d, sizeof(double) * o->d);
        memcpy(u->V + (size_t)u->len * o->d, v + (size_t)h * o->d, sizeof(double) * o->d);
        u->S[u->len] = 0.0;
        u->C[u->len] = 0;
        u->pos[u->len] = o->n_seen[b];
        u->len += 1;
    }
    o->n_seen[b] += 1;
}

/* Section 4.1 "Position Encoding": in-cache positions.  Tables by slot; cos/sin are single-precision inputs. */
int tkvo_set_rope(tkvo *o, const float *cos_tab, const float *sin_tab, int slots, int round_bf16) {
    if (o->d % 2 || o->d > 512) return -1;
    o->rope_cos = cos_tab; o->rope_sin = sin_tab; o->rope_slots = cos_tab ? slots : 0; o->rope_round_bf16 = round_bf16;
    return 0;
}

static float round_to_bf16(float x) { /* round to nearest even to 8 significand bits, kept in a float */
    uint32_t u;
    memcpy(&u, &x, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return x;
    u += 0x7fffu + ((u >> 16) & 1u);
    u &= 0xffff0000u;
    memcpy(&x, &u, 4);
    return x;
}

/* x (an element-type value held in a double) rotated to slot `slot`: pairs (t, t + d/2), two single-precision
 * operations per output, then rounded to the cache's element type. */
static void rope_row(const tkvo *o, const double *x, int slot, double *y) {
    const int half = o->d / 2;
    const float *cs = o->rope_cos + (size_t)slot * half, *sn = o->rope_sin + (size_t)slot * half;
    for (int t = 0; t < half; ++t) {
        const float x1 = (float)x[t], x2 = (float)x[t + half];
        volatile float p1 = x2 * sn[t], p2 = x1 * sn[t]; /* each product rounded to single precision */
        float y1 = fmaf(x1, cs[t], -p1), y2 = fmaf(x2, cs[t], p2);
        if (o->rope_round_bf16) { y1 = round_to_bf16(y1); y2 = round_to_bf16(y2); }
        y[t] = (double)y1; y[t + half] = (double)y2;
    }
}

/* One query row against one unit: a = SoftMax(q K^T / sqrt(d)) over the first
 * n_vis slots (Section 3.1), out = a V.  a is returned in prob[0..n_vis).
 * With in-cache positions the query is encoded at slot n_vis - 1 (its own) and key j at slot j. */
static void attend_row(const tkvo *o, const tkvo_unit *u, const double *q_in, int n_vis, double *prob, double *out) {
    const int d = o->d;
    const double inv = 1.0 / sqrt((double)d);
    double mx = -INFINITY;
    double qbuf[512], kbuf[512];
    const double *q = q_in;
    if (o->rope_cos) { rope_row(o, q_in, n_vis - 1, qbuf); q = qbuf; }
    for (int j = 0; j < n_vis; ++j) {
        double s = 0.0;
        const double *kj = u->K + (size_t)j * d;
        if (o->rope_cos) { rope_row(o, kj, j, kbuf); kj = kbuf; }
        for (int t = 0; t < d; ++t) s += q[t] * kj[t];
        s *= inv;
        prob[j] = s;
        if (s > mx) mx = s;
    }
    double den = 0.0;
    for (int j = 0; j < n_vis; ++j) { prob[j] = exp(prob[j] - mx); den += prob[j]; }
    for (int j = 0; j < n_vis; ++j) prob[j] /= den;
    for (int t = 0; t < d; ++t) out[t] = 0.0;
    for (int j = 0; j < n_vis; ++j) {
        const double *vj = u->V + (size_t)j * d;
        const double a = prob[j];
        for (int t = 0; t < d; ++t) out[t] += a * vj[t];
    }
}

/*
 * Decode, first half (Alg. 1, loop body up to the S update): append, attend, advance C and S.
 * q,out: [B][Hq][d]; k,v: [B][Hkv][d]; active: [B] or NULL (all active).
 */
void tkvo_decode_attend(tkvo *o, const double *q, const double *k, const double *v, double *out,
                        const uint8_t *active) {
    const int d = o->d, g = o->g;
    for (int b = 0; b < o->B; ++b) {
        if (active && !active[b]) continue;
        append_token(o, b, k + (size_t)b * o->Hkv * d, v + (size_t)b * o->Hkv * d);
    }
#pragma omp parallel for schedule(dynamic)
    for (int bu = 0; bu < o->B * o->Hkv; ++bu) {
        const int b = bu / o->Hkv, kh = bu % o->Hkv;
        if (active && !active[b]) continue;
        tkvo_unit *u = &o->u[bu];
        double *prob = (double *)malloc(sizeof(double) * (size_t)u->len);
        double *acc = (double *)calloc((size_t)u->len, sizeof(double));
        for (int hh = 0; hh < g; ++hh) {
            const int h = kh * g + hh;
            attend_row(o, u, q + ((size_t)b * o->Hq + h) * d, u->len, prob, out + ((size_t)b * o->Hq + h) * d);
            for (int j = 0; j < u->len; ++j) acc[j] += prob[j];
        }
        for (int j = 0; j < u->len; ++j) {
            u->C[j] += 1;               /* Alg. 1: C <- (C u {0}) + 1 */
            u->S[j] += acc[j] / (double)g; /* Alg. 1: S <- (S u {0}) + a, group mean */
        }
        free(prob); free(acc);
    }
}

/*
 * Chunked prefill, first half: append chunk_lens[b] tokens of sequence b, each
 * chunk row attends causally, C and S advance by the whole chunk.
 * q,out: [B][stride][Hq][d]; k,v: [B][stride][Hkv][d]; chunk_lens: [B] (0 = skip).
 */
void tkvo_prefill_attend(tkvo *o, const double *q, const double *k, const double *v, double *out,
                         const int32_t *chunk_lens, int stride) {
    const int d = o->d, g = o->g;
    for (int b = 0; b < o->B; ++b) {
        for (int i = 0; i < chunk_lens[b]; ++i) {
            const size_t row = (size_t)b * stride + i;
            append_token(o, b, k + row * o->Hkv * d, v + row * o->Hkv * d);
        }
    }
#pragma omp parallel for schedule(dynamic)
    for (int bu = 0; bu < o->B * o->Hkv; ++bu) {
        const int b = bu / o->Hkv, kh = bu % o->Hkv;
        const int m = chunk_lens[b];
        if (m <= 0) continue;
        tkvo_unit *u = &o->u[bu];
        const int n = u->len;
        double *prob = (double *)malloc(sizeof(double) * (size_t)n);
        double *acc = (double *)calloc((size_t)n, sizeof(double));
        for (int i = 0; i < m; ++i) {
            /* chunk token i sits in slot n-m+i; it sees slots 0..n-m+i (pos <= its own) */
            const int n_vis = n - m + i + 1;
            for (int hh = 0; hh < g; ++hh) {
                const int h = kh * g + hh;
                const size_t qo = (((size_t)b * stride + i) * o->Hq + h) * d;
                attend_row(o, u, q + qo, n_vis, prob, out + qo);
                for (int j = 0; j < n_vis; ++j) acc[j] += prob[j];
            }
            for (int j = 0; j < n_vis; ++j) u->C[j] += 1; /* one "step" per chunk row */
        }
        for (int j = 0; j < n; ++j) u->S[j] += acc[j] / (double)g;
        free(prob); free(acc);
    }
}

static void unit_remove(tkvo_unit *u, int d, int slot) { /* 0-based slot, order preserved */
    const int tail = u->len - slot - 1;
    memmove(u->K + (size_t)slot * d, u->K + (size_t)(slot + 1) * d, sizeof(double) * (size_t)tail * d);
    memmove(u->V + (size_t)slot * d, u->V + (size_t)(slot + 1) * d, sizeof(double) * (size_t)tail * d);
    memmove(u->S + slot, u->S + slot + 1, sizeof(double) * (size_t)tail);
    memmove(u->C + slot, u->C + slot + 1, sizeof(int64_t) * (size_t)tail);
    memmove(u->pos + slot, u->pos + slot + 1, sizeof(int64_t) * (size_t)tail);
    u->len -= 1;
}

static int in_sorted(const int32_t *a, int n, int64_t x) {
    int lo = 0, hi = n;
    while (lo < hi) { int mid = (lo + hi) / 2; if (a[mid] < x) lo = mid + 1; else hi = mid; }
    return lo < n && a[lo] == x;
}

/*
 * One-shot prefill, first half (Section 4.2): the whole prompt of lens[b] tokens enters an empty cache, every
 * row attends causally (the output is plain attention over the prompt), and the last `block` rows - the
 * observation window - advance S and C of every token they see (Algorithm 1's two update lines, for those
 * rows only).  lens[b] must be a multiple of `block`; sequences with lens[b] = 0 are skipped.
 * Returns 0, or -1 on a bad argument / non-empty cache.
 */
int tkvo_prefill_oneshot_attend(tkvo *o, const double *q, const double *k, const double *v, double *out,
                                const int32_t *lens, int stride, int block) {
    const int d = o->d, g = o->g;
    if (block < 1 || o->c % block || o->n_sink || o->n_recent) return -1;
    for (int b = 0; b < o->B; ++b)
        if (lens[b] < 0 || lens[b] > stride || lens[b] % block || (lens[b] && o->n_seen[b])) return -1;
    for (int b = 0; b < o->B; ++b) {
        for (int i = 0; i < lens[b]; ++i) {
            const size_t row = (size_t)b * stride + i;
            append_token(o, b, k + row * o->Hkv * d, v + row * o->Hkv * d);
        }
        if (lens[b]) o->pending_block[b] = block;
    }
#pragma omp parallel for schedule(dynamic)
    for (int bu = 0; bu < o->B * o->Hkv; ++bu) {
        const int b = bu / o->Hkv, kh = bu % o->Hkv;
        const int T = lens[b];
        if (T <= 0) continue;
        tkvo_unit *u = &o->u[bu];
        double *prob = (double *)malloc(sizeof(double) * (size_t)T);
        double *acc = (double *)calloc((size_t)T, sizeof(double));
        for (int i = 0; i < T; ++i) {
            const int in_window = (i >= T - block);
            for (int hh = 0; hh < g; ++hh) {
                const int h = kh * g + hh;
                const size_t qo = (((size_t)b * stride + i) * o->Hq + h) * d;
                attend_row(o, u, q + qo, i + 1, prob, out + qo);
                if (in_window) for (int j = 0; j <= i; ++j) acc[j] += prob[j];
            }
            if (in_window) for (int j = 0; j <= i; ++j) u->C[j] += 1; /* Alg. 1: C <- C + 1, window rows only */
        }
        for (int j = 0; j < T; ++j) u->S[j] += acc[j] / (double)g;    /* Alg. 1: S <- S + a, group mean */
        free(prob); free(acc);
    }
    return 0;
}

/*
 * One-shot prefill, second half (Section 4.2, "Block-level Eviction"): a block's score is the mean of its
 * tokens' S / C; blocks enter a cache of c / block blocks in order and Algorithm 1's "length > c" branch plays
 * on blocks.  Near-ties and hints as in tkvo_evict (a block is "in the hint" when its first token is).
 */
void tkvo_evict_blocks(tkvo *o, const int32_t *hint_pos, const int32_t *hint_cnt, double near_tie_tol) {
    o->last_near_ties = 0; o->last_hint_flips = 0; o->last_min_gap = INFINITY;
    const int c = o->c, d = o->d;
    for (int b = 0; b < o->B; ++b) {
        const int bs = o->pending_block[b];
        if (!bs) continue;
        o->pending_block[b] = 0;
        const int T = o->u[b * o->Hkv].len, nb = T / bs, cb = c / bs;
        int idx_end = 1;
        for (int kh = 0; kh < o->Hkv; ++kh) {
            tkvo_unit *u = &o->u[b * o->Hkv + kh];
            double *score = (double *)malloc(sizeof(double) * (size_t)nb);
            for (int kb = 0; kb < nb; ++kb) { /* averaged importance of the b tokens of the block */
                double a = 0.0;
                for (int t = 0; t < bs; ++t)
                    a += o->rule == TKVO_RULE_ACCUMULATED ? u->S[kb * bs + t] : u->S[kb * bs + t] / (double)u->C[kb * bs + t];
                score[kb] = a / (double)bs;
            }
            int *cache = (int *)malloc(sizeof(int) * (size_t)(cb + 1)); /* block numbers, in order */
            int len = 0, idx = 1;
            for (int kb = 0; kb < nb; ++kb) {
                cache[len++] = kb; /* the block arrives */
                if (len > cb) {
                    const int l = idx - 1, r = idx;
                    int evict_right;
                    if (o->rule == TKVO_RULE_KEEP_LEFT) evict_right = 1;
                    else if (o->rule == TKVO_RULE_EVICT_LEFT) evict_right = 0;
                    else {
                        const double sl = score[cache[l]], sr = score[cache[r]];
                        evict_right = (sl > sr); /* Alg. 1: strict > */
                        const double mxabs = fmax(fabs(sl), fabs(sr));
                        const double gap = mxabs > 0.0 ? fabs(sl - sr) / mxabs : 0.0;
                        if (gap < o->last_min_gap) o->last_min_gap = gap;
                        if (gap < near_tie_tol) {
                            o->last_near_ties += 1;
                            if (hint_pos) {
                                const int32_t *hp = hint_pos + ((size_t)b * o->Hkv + kh) * c;
                                const int hn = hint_cnt[b * o->Hkv + kh];
                                const int lin = in_sorted(hp, hn, u->pos[cache[l] * bs]);
                                const int rin = in_sorted(hp, hn, u->pos[cache[r] * bs]);
                                if (lin != rin) {
                                    const int want = lin ? 1 : 0;
                                    if (want != evict_right) { evict_right = want; o->last_hint_flips += 1; }
                                }
                            }
                        }
                    }
                    const int gone = evict_right ? r : l;
                    memmove(cache + gone, cache + gone + 1, sizeof(int) * (size_t)(len - gone - 1));
                    len -= 1;
                    idx = (idx % cb) + 1;
                }
            }
            /* keep the tokens of the surviving blocks, in order */
            int w = 0;
            for (int s = 0; s < len; ++s) {
                for (int t = 0; t < bs; ++t, ++w) {
                    const int src = cache[s] * bs + t;
                    if (src == w) continue;
                    memcpy(u->K + (size_t)w * d, u->K + (size_t)src * d, sizeof(double) * d);
                    memcpy(u->V + (size_t)w * d, u->V + (size_t)src * d, sizeof(double) * d);
                    u->S[w] = u->S[src]; u->C[w] = u->C[src]; u->pos[w] = u->pos[src];
                }
            }
            u->len = w;
            idx_end = idx;
            free(score); free(cache);
        }
        if (T > c) {
            o->n_evicted[b] += T - c;
            o->idx[b] = (idx_end - 1) * bs + 1; /* the first token of the block the block pointer stands on */
        }
    }
    o->total_near_ties += o->last_near_ties;
    o->total_hint_flips += o->last_hint_flips;
}

/*
 * Second half (Alg. 1, the "length > c" branch), repeated while the cache is longer than c.
 * Scores are not touched by eviction, so repeating the branch uses frozen
 * averaged scores.  idx advances once per eviction round of a sequence (all
 * KV heads of a sequence have the same length, hence the same idx).
 *
 * Near-ties: a decision whose relative gap |a-b|/max(|a|,|b|) is below
 * near_tie_tol is counted.  If hint_pos/hint_cnt are given ([B][Hkv][c] sorted
 * positions another implementation retained, and their counts), a near-tie
 * decision follows the hint when exactly one member of the pair is in it; the
 * number of decisions changed this way is reported.  Decisions that are not
 * near-ties never look at the hint.
 */
void tkvo_evict(tkvo *o, const int32_t *hint_pos, const int32_t *hint_cnt, double near_tie_tol) {
    o->last_near_ties = 0; o->last_hint_flips = 0; o->last_min_gap = INFINITY;
    const int c = o->c, d = o->d;
    const int c_mid = c - o->n_sink - o->n_recent; /* size of the region Algorithm 1 runs on (= c without protection) */
    for (int b = 0; b < o->B; ++b) {
        while (o->u[b * o->Hkv].len > c) {
            const int idx = o->idx[b]; /* 1-based within the middle region: scope is its slots idx, idx+1 */
            for (int kh = 0; kh < o->Hkv; ++kh) {
                tkvo_unit *u = &o->u[b * o->Hkv + kh];
                const int l = o->n_sink + idx - 1, r = o->n_sink + idx; /* 0-based slots of the whole cache */
                int evict_right;
                if (o->rule == TKVO_RULE_KEEP_LEFT) evict_right = 1;
                else if (o->rule == TKVO_RULE_EVICT_LEFT) evict_right = 0;
                else {
                    const int acc = o->rule == TKVO_RULE_ACCUMULATED;
                    const double sl = acc ? u->S[l] : u->S[l] / (double)u->C[l]; /* Alg. 1: S-bar = S / C */
                    const double sr = acc ? u->S[r] : u->S[r] / (double)u->C[r];
                    evict_right = (sl > sr);                      /* Alg. 1: strict > */
                    const double mxabs = fmax(fabs(sl), fabs(sr));
                    const double gap = mxabs > 0.0 ? fabs(sl - sr) / mxabs : 0.0;
                    if (gap < o->last_min_gap) o->last_min_gap = gap;
                    if (gap < near_tie_tol) {
                        o->last_near_ties += 1;
                        if (hint_pos) {
                            const int32_t *hp = hint_pos + ((size_t)b * o->Hkv + kh) * c;
                            const int hn = hint_cnt[b * o->Hkv + kh];
                            const int lin = in_sorted(hp, hn, u->pos[l]);
                            const int rin = in_sorted(hp, hn, u->pos[r]);
                            if (lin != rin) {
                                const int want = lin ? 1 : 0; /* keep the one in the hint */
                                if (want != evict_right) { evict_right = want; o->last_hint_flips += 1; }
                            }
                        }
                    }
                }
                unit_remove(u, d, evict_right ? r : l); /* Alg. 1: evict one of the pair */
            }
            if (o->idx_mode == TKVO_IDX_LITERAL) o->idx[b] = (idx + 1) % c_mid + 1;
            else o->idx[b] = (idx % c_mid) + 1; /* idx update, as the prose of Section 4.1 reads */
            o->n_evicted[b] += 1;
        }
    }
    o->total_near_ties += o->last_near_ties;
    o->total_hint_flips += o->last_hint_flips;
}

void tkvo_decode_step(tkvo *o, const double *q, const double *k, const double *v, double *out,
                      const uint8_t *active) {
    tkvo_decode_attend(o, q, k, v, out, active);
    tkvo_evict(o, NULL, NULL, 1e-4);
}

void tkvo_prefill_chunk(tkvo *o, const double *q, const double *k, const double *v, double *out,
                        const int32_t *chunk_lens, int stride) {
    tkvo_prefill_attend(o, q, k, v, out, chunk_lens, stride);
    tkvo_evict(o, NULL, NULL, 1e-4);
}

/* ---- read-outs ---- */
int tkvo_len(const tkvo *o, int b, int kh) { return o->u[b * o->Hkv + kh].len; }
int64_t tkvo_n_seen(const tkvo *o, int b) { return o->n_seen[b]; }
int64_t tkvo_n_evicted(const tkvo *o, int b) { return o->n_evicted[b]; }
int tkvo_idx(const tkvo *o, int b) { return o->idx[b]; }
int64_t tkvo_last_near_ties(const tkvo *o) { return o->last_near_ties; }
int64_t tkvo_last_hint_flips(const tkvo *o) { return o->last_hint_flips; }
double tkvo_last_min_gap(const tkvo *o) { return o->last_min_gap; }
int64_t tkvo_total_near_ties(const tkvo *o) { return o->total_near_ties; }
int64_t tkvo_total_hint_flips(const tkvo *o) { return o->total_hint_flips; }

/* positions, raw S, C, averaged score S/C of unit (b,kh); each array holds >= len entries */
int tkvo_read_unit(const tkvo *o, int b, int kh, int64_t *pos, double *S, int64_t *C, double *sbar) {
    const tkvo_unit *u = &o->u[b * o->Hkv + kh];
    for (int j = 0; j < u->len; ++j) {
        if (pos) pos[j] = u->pos[j];
        if (S) S[j] = u->S[j];
        if (C) C[j] = u->C[j];
        if (sbar) sbar[j] = u->S[j] / (double)u->C[j];
    }
    return u->len;
}

/* cached keys / values of a unit, [len][d] */
int tkvo_read_kv(const tkvo *o, int b, int kh, double *K, double *V) {
    const tkvo_unit *u = &o->u[b * o->Hkv + kh];
    if (K) memcpy(K, u->K, sizeof(double) * (size_t)u->len * o->d);
    if (V) memcpy(V, u->V, sizeof(double) * (size_t)u->len * o->d);
    return u->len;
}
