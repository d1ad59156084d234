/*
 * corm_oracle.c — TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of what the CORM hot path computes, written from the paper:
 *   - scaled dot-product attention for one decode query per head            (Eq. 1)
 *   - the normalised attention score alpha_{t,i}                             (Eq. 2)
 *   - "important key": alpha_{t,i} >= threshold, threshold = alpha_scale/t   (Definition 3.1)
 *   - "long-term minor key": minor for every one of the recent w queries     (Definition 4.1, Approach paragraph)
 *   - the eviction step with warm-up and recent-r protection                 (Algorithm 1)
 *   - the grouped-query rule: a shared KV head drops a key only when every
 *     query head of its group judged it minor in all recent queries          (Section 5, "Integrate into GQA")
 *   - a prompt-end pass that applies the same rule to the causal attention
 *     rows of the last w prompt queries (the paper only covers generation;
 *     the zero-padding of Algorithm 1 fixes the bits of keys newer than a query).
 *
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may use this file.
 * It shares no code with the CUDA library and never calls it.
 *
 * The recent-w verdict rows of Algorithm 1 (a bool matrix [m, l]) are held here as one w-bit shift register per
 * key (REG_WORDS 32-bit words, w <= 256): bit b of a key's register is the verdict of the query b steps ago. A
 * second statement of the policy with another data structure (per key, the set of queries that found it
 * important) lives in verdict_history.py and is tested equal to this one.
 *
 * Every function below is pinned by tests/test_oracle_pins.py (hand-worked cases, full attention at alpha=0,
 * brute force over subsets, closed forms, invariants); none is "parity unpinned".
 *
 * State of one unit (layer, sequence, kv head): an ordered list of live entries (pos, k[d], v[d], word).
 * State of one (layer, sequence): t = tokens seen so far, n_obs = verdict rows recorded (<= w).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
    int n_layers, batch, n_q_heads, n_kv_heads, head_dim, max_tokens, w, r;
    double alpha;
    int     *live;   /* [L*B*Hkv]            live entries per unit            */
    int     *pos;    /* [L*B*Hkv][C]         absolute 1-based token position  */
    uint32_t *word;  /* [L*B*Hkv][C][REG_WORDS] w-bit verdict register (word 0 = newest 32 verdicts) */
    double  *k, *v;  /* [L*B*Hkv][C][d]                                       */
    int     *t;      /* [L*B]                tokens seen                      */
    int     *n_obs;  /* [L*B]                verdict rows recorded            */
    long long appended, evicted, verdict_evals, near_threshold;
    double *q_prev;      /* [n_layers][batch][n_q_heads][d]: the previous decode step's queries */
    unsigned char *has_prev; /* [n_layers] */
    double sim_sum; long long sim_count; /* Eq. 3 between each head's query and its previous one */
    long long important, judged; /* decode steps only: keys judged important / keys judged (the sparsity of Section 3.1) */
    double  near_rel; /* half-width of the reported band around the threshold, relative */
} corm_oracle;

enum { ORACLE_OK = 0, ORACLE_BAD_ARG = 1, ORACLE_CAPACITY = 6 };
enum { REG_WORDS = 8, MAX_WINDOW = 32 * REG_WORDS };

static size_t unit_index(const corm_oracle *o, int layer, int b, int h) {
    return ((size_t)layer * o->batch + b) * o->n_kv_heads + h;
}

corm_oracle *oracle_create(int n_layers, int batch, int n_q_heads, int n_kv_heads, int head_dim, int max_tokens,
                           int w, int r, double alpha) {
    if (n_layers < 1 || batch < 1 || n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads) return NULL;
    if (head_dim < 1 || max_tokens < 1 || w < 1 || w > MAX_WINDOW || r < 1 || !(alpha >= 0.0)) return NULL;
    corm_oracle *o = (corm_oracle *)calloc(1, sizeof(corm_oracle));
    if (!o) return NULL;
    o->n_layers = n_layers; o->batch = batch; o->n_q_heads = n_q_heads; o->n_kv_heads = n_kv_heads;
    o->head_dim = head_dim; o->max_tokens = max_tokens; o->w = w; o->r = r; o->alpha = alpha;
    o->near_rel = 1e-6;
    size_t units = (size_t)n_layers * batch * n_kv_heads, C = (size_t)max_tokens, d = (size_t)head_dim;
    o->live = (int *)calloc(units, sizeof(int));
    o->pos = (int *)calloc(units * C, sizeof(int));
    o->word = (uint32_t *)calloc(units * C * REG_WORDS, sizeof(uint32_t));
    o->k = (double *)calloc(units * C * d, sizeof(double));
    o->v = (double *)calloc(units * C * d, sizeof(double));
    o->t = (int *)calloc((size_t)n_layers * batch, sizeof(int));
    o->n_obs = (int *)calloc((size_t)n_layers * batch, sizeof(int));
    o->q_prev = (double *)calloc((size_t)n_layers * batch * n_q_heads * d, sizeof(double));
    o->has_prev = (unsigned char *)calloc((size_t)n_layers, 1);
    if (!o->live || !o->pos || !o->word || !o->k || !o->v || !o->t || !o->n_obs || !o->q_prev || !o->has_prev) return NULL;
    return o;
}

void oracle_destroy(corm_oracle *o) {
    if (!o) return;
    free(o->live); free(o->pos); free(o->word); free(o->k); free(o->v); free(o->t); free(o->n_obs); free(o->q_prev); free(o->has_prev); free(o);
}

/* register helpers: shift the newest verdict in at bit 0 and drop everything older than w verdicts */
static void reg_shift_in(uint32_t *reg, int w, uint32_t bit) {
    uint32_t carry = bit & 1u;
    for (int i = 0; i < REG_WORDS; ++i) {
        uint32_t next = reg[i] >> 31;
        reg[i] = (reg[i] << 1) | carry;
        carry = next;
    }
    for (int i = 0; i < REG_WORDS; ++i) {            /* keep bits [0, w) */
        int lo = 32 * i;
        if (w <= lo) reg[i] = 0u;
        else if (w < lo + 32) reg[i] &= (1u << (w - lo)) - 1u;
    }
}
static int reg_nonzero(const uint32_t *reg) {
    for (int i = 0; i < REG_WORDS; ++i) if (reg[i]) return 1;
    return 0;
}
static void reg_clear(uint32_t *reg) { memset(reg, 0, REG_WORDS * sizeof(uint32_t)); }

/* Algorithm 1, the part after the message update: once w rows are recorded, a key stays iff some recent query
 * found it important (any over the window) or it is one of the r most recent tokens; survivors keep their order
 * and their message columns move with them. t is the absolute token count of the sequence.
 * Returns the number of entries discarded. */
static int evict_unit(corm_oracle *o, size_t u, int t, int n_obs) {
    if (n_obs < o->w) return 0; /* warm-up: fewer than w verdict rows, nothing is discarded */
    size_t C = (size_t)o->max_tokens, d = (size_t)o->head_dim;
    int l = o->live[u], kept = 0;
    for (int j = 0; j < l; ++j) {
        int keep = reg_nonzero(o->word + (u * C + j) * REG_WORDS) || (o->pos[u * C + j] > t - o->r);
        if (!keep) continue;
        if (kept != j) {
            o->pos[u * C + kept] = o->pos[u * C + j];
            memcpy(o->word + (u * C + kept) * REG_WORDS, o->word + (u * C + j) * REG_WORDS, REG_WORDS * sizeof(uint32_t));
            memcpy(o->k + (u * C + kept) * d, o->k + (u * C + j) * d, d * sizeof(double));
            memcpy(o->v + (u * C + kept) * d, o->v + (u * C + j) * d, d * sizeof(double));
        }
        ++kept;
    }
    o->live[u] = kept;
    return l - kept;
}

/* One softmax row (Eq. 2) of query qv over the first n live keys of unit u. With limit_pos >= 0 only entries whose
 * position is <= limit_pos take part (a causal prompt row); the others get p = 0. */
static void softmax_row(const corm_oracle *o, size_t u, const double *qv, int n, int limit_pos, double *p) {
    size_t C = (size_t)o->max_tokens, d = (size_t)o->head_dim;
    double root_d = sqrt((double)o->head_dim), m = -INFINITY, Z = 0.0;
    for (int j = 0; j < n; ++j) {
        if (limit_pos >= 0 && o->pos[u * C + j] > limit_pos) continue;
        const double *kj = o->k + (u * C + j) * d;
        double s = 0.0;
        for (size_t c = 0; c < d; ++c) s += qv[c] * kj[c];
        p[j] = s / root_d;
        if (p[j] > m) m = p[j];
    }
    for (int j = 0; j < n; ++j) {
        if (limit_pos >= 0 && o->pos[u * C + j] > limit_pos) continue;
        p[j] = exp(p[j] - m);
        Z += p[j];
    }
    for (int j = 0; j < n; ++j) {
        if (limit_pos >= 0 && o->pos[u * C + j] > limit_pos) p[j] = 0.0;
        else p[j] /= Z;
    }
}

/* Definition 3.1 with the scale parameter: important iff p >= alpha/t. Also counts evaluations that fall inside
 * the reported band |p - thr| <= near_rel * thr (no band when the threshold is 0). */
static int important(const corm_oracle *o, double p, int t, long long *evals, long long *near) {
    double thr = o->alpha / (double)t;
    ++*evals;
    if (thr > 0.0 && fabs(p - thr) <= o->near_rel * thr) ++*near;
    return p >= thr;
}

/* Decode step for every unit of one layer.
 * q [B,Hq,d], k_new/v_new [B,Hkv,d], out [B,Hq,d] (inputs are float: exact carriers of the cache dtype's values).
 * imp_out (optional) [B,Hkv,C] bytes: the OR-ed verdict of this step for each live slot before eviction. */
int oracle_decode_step(corm_oracle *o, int layer, const float *q, const float *k_new, const float *v_new,
                       double *out, unsigned char *imp_out) {
    if (!o || layer < 0 || layer >= o->n_layers || !q || !k_new || !v_new || !out) return ORACLE_BAD_ARG;
    const int B = o->batch, Hq = o->n_q_heads, Hkv = o->n_kv_heads, G = Hq / Hkv, d = o->head_dim;
    const size_t C = (size_t)o->max_tokens;
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < Hkv; ++h)
            if (o->live[unit_index(o, layer, b, h)] + 1 > o->max_tokens) return ORACLE_CAPACITY;
    /* Eq. 3: cosine similarity of every query head's query with the one of the previous decode step (Section 3.3
     * observes that the current query is most similar to recent ones); heads with a zero vector are skipped */
    {
        double *prev = o->q_prev + (size_t)layer * B * Hq * d;
        for (int x = 0; x < B * Hq; ++x) {
            if (o->has_prev[layer]) {
                double dot = 0.0, n1 = 0.0, n2 = 0.0;
                for (int c = 0; c < d; ++c) {
                    double a = (double)q[(size_t)x * d + c], pb = prev[(size_t)x * d + c];
                    dot += a * pb; n1 += a * a; n2 += pb * pb;
                }
                if (n1 > 0.0 && n2 > 0.0) { o->sim_sum += dot / (sqrt(n1) * sqrt(n2)); o->sim_count += 1; }
            }
            for (int c = 0; c < d; ++c) prev[(size_t)x * d + c] = (double)q[(size_t)x * d + c];
        }
        o->has_prev[layer] = 1;
    }
    long long evals_total = 0, near_total = 0, appended = 0, evicted = 0, important_total = 0, judged_total = 0;
#pragma omp parallel for collapse(2) schedule(dynamic) reduction(+ : evals_total, near_total, appended, evicted, important_total, judged_total)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hkv; ++h) {
            size_t u = unit_index(o, layer, b, h);
            int t = o->t[(size_t)layer * B + b] + 1;
            int n_obs = o->n_obs[(size_t)layer * B + b] + 1 < o->w ? o->n_obs[(size_t)layer * B + b] + 1 : o->w;
            /* append the current token: Algorithm 1's keys [l, d] include it, its message column is zero */
            int l = o->live[u];
            for (int c = 0; c < d; ++c) {
                o->k[(u * C + l) * d + c] = (double)k_new[((size_t)b * Hkv + h) * d + c];
                o->v[(u * C + l) * d + c] = (double)v_new[((size_t)b * Hkv + h) * d + c];
            }
            o->pos[u * C + l] = t;
            reg_clear(o->word + (u * C + l) * REG_WORDS);
            l += 1;
            o->live[u] = l;
            ++appended;
            double *p = (double *)malloc((size_t)l * sizeof(double));
            double *qv = (double *)malloc((size_t)d * sizeof(double));
            unsigned char *imp = (unsigned char *)calloc((size_t)l, 1);
            long long evals = 0, near = 0;
            for (int g = 0; g < G; ++g) {
                size_t qh = (size_t)b * Hq + (size_t)h * G + g;
                for (int c = 0; c < d; ++c) qv[c] = (double)q[qh * d + c];
                softmax_row(o, u, qv, l, -1, p);
                for (int c = 0; c < d; ++c) {                       /* Eq. 1: out = sum_j p_j v_j */
                    double acc = 0.0;
                    for (int j = 0; j < l; ++j) acc += p[j] * o->v[(u * C + j) * d + c];
                    out[qh * d + c] = acc;
                }
                for (int j = 0; j < l; ++j)                           /* group rule: OR over the query heads */
                    if (important(o, p[j], t, &evals, &near)) imp[j] = 1;
            }
            for (int j = 0; j < l; ++j) {                             /* newest verdict enters at bit 0 */
                reg_shift_in(o->word + (u * C + j) * REG_WORDS, o->w, (uint32_t)imp[j]);
                if (imp_out) imp_out[((size_t)b * Hkv + h) * C + j] = imp[j];
                important_total += imp[j];
            }
            judged_total += l;
            evals_total += evals; near_total += near;
            free(p); free(qv); free(imp);
            evicted += evict_unit(o, u, t, n_obs);                    /* Algorithm 1's eviction, effective next step */
        }
    }
    for (int b = 0; b < B; ++b) {
        size_t s = (size_t)layer * B + b;
        o->t[s] += 1;
        o->n_obs[s] = o->n_obs[s] + 1 < o->w ? o->n_obs[s] + 1 : o->w;
    }
    o->evicted += evicted;
    o->appended += appended;
    o->verdict_evals += evals_total;
    o->near_threshold += near_total;
    o->important += important_total;
    o->judged += judged_total;
    return ORACLE_OK;
}

/* Section 3.1's sparsity over the decode steps so far: keys judged important (Definition 3.1, OR over the group)
 * and keys judged. */
void oracle_sparsity(const corm_oracle *o, long long *important, long long *judged) {
    if (important) *important = o->important;
    if (judged) *judged = o->judged;
}

/* Sum and number of the adjacent-query cosine similarities (Eq. 3) over the decode steps so far. */
void oracle_similarity(const corm_oracle *o, double *sum, long long *count) {
    if (sum) *sum = o->sim_sum;
    if (count) *count = o->sim_count;
}

/* Prompt-end pass for every unit of one layer.
 * k_prompt/v_prompt [B,Hkv,p_max,d]; q_last [B,Hq,w,d] = queries of prompt positions P-w+1..P, oldest first (for
 * P < w the first w-P rows are ignored); prompt_lens [B]. All P keys enter the cache, then the causal attention
 * row of each of the last min(P,w) prompt queries, taken over the full prompt, is recorded exactly as a decode
 * step would record it (threshold alpha/i for the query at position i; keys newer than the query get a 0 bit),
 * and one eviction with t = P follows. */
int oracle_compress_prompt(corm_oracle *o, int layer, const float *k_prompt, const float *v_prompt,
                           const float *q_last, const int *prompt_lens, int p_max) {
    if (!o || layer < 0 || layer >= o->n_layers || !prompt_lens || p_max < 0) return ORACLE_BAD_ARG;
    const int B = o->batch, Hq = o->n_q_heads, Hkv = o->n_kv_heads, G = Hq / Hkv, d = o->head_dim, w = o->w;
    const size_t C = (size_t)o->max_tokens;
    for (int b = 0; b < B; ++b) {
        if (prompt_lens[b] < 0 || prompt_lens[b] > p_max) return ORACLE_BAD_ARG;
        if (prompt_lens[b] > o->max_tokens) return ORACLE_CAPACITY;
        if (prompt_lens[b] > 0 && (!k_prompt || !v_prompt || !q_last)) return ORACLE_BAD_ARG;
    }
    o->has_prev[layer] = 0;                 /* a new prompt: the layer's previous decode query belongs to the old text */
    long long evals_total = 0, near_total = 0, appended = 0, evicted = 0;
#pragma omp parallel for collapse(2) schedule(dynamic) reduction(+ : evals_total, near_total, appended, evicted)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hkv; ++h) {
            size_t u = unit_index(o, layer, b, h);
            int P = prompt_lens[b], wp = P < w ? P : w;
            for (int j = 0; j < P; ++j) {
                size_t src = (((size_t)b * Hkv + h) * (size_t)p_max + j) * d;
                for (int c = 0; c < d; ++c) {
                    o->k[(u * C + j) * d + c] = (double)k_prompt[src + c];
                    o->v[(u * C + j) * d + c] = (double)v_prompt[src + c];
                }
                o->pos[u * C + j] = j + 1;
                reg_clear(o->word + (u * C + j) * REG_WORDS);
            }
            o->live[u] = P;
            appended += P;
            if (P == 0) continue;
            double *p = (double *)malloc((size_t)P * sizeof(double));
            double *qv = (double *)malloc((size_t)d * sizeof(double));
            unsigned char *imp = (unsigned char *)malloc((size_t)P);
            long long evals = 0, near = 0;
            for (int row = w - wp; row < w; ++row) {
                int i = P - (w - 1 - row);                            /* absolute position of this query */
                memset(imp, 0, (size_t)P);
                for (int g = 0; g < G; ++g) {
                    size_t qh = ((size_t)b * Hq + (size_t)h * G + g) * (size_t)w + row;
                    for (int c = 0; c < d; ++c) qv[c] = (double)q_last[qh * d + c];
                    softmax_row(o, u, qv, P, i, p);                   /* causal: keys 1..i only */
                    for (int j = 0; j < i; ++j)                       /* slot j holds position j+1 here */
                        if (important(o, p[j], i, &evals, &near)) imp[j] = 1;
                }
                for (int j = 0; j < P; ++j) reg_shift_in(o->word + (u * C + j) * REG_WORDS, w, (uint32_t)imp[j]);
            }
            free(p); free(qv); free(imp);
            evals_total += evals; near_total += near;
            evicted += evict_unit(o, u, P, wp);
        }
    }
    for (int b = 0; b < B; ++b) {
        size_t s = (size_t)layer * B + b;
        o->t[s] = prompt_lens[b];
        o->n_obs[s] = prompt_lens[b] < w ? prompt_lens[b] : w;
    }
    o->appended += appended; o->evicted += evicted;
    o->verdict_evals += evals_total; o->near_threshold += near_total;
    return ORACLE_OK;
}

/* ---- state access (tests, lockstep parity) ---- */

int oracle_live_len(const corm_oracle *o, int layer, int b, int h) { return o->live[unit_index(o, layer, b, h)]; }
int oracle_n_tokens(const corm_oracle *o, int layer, int b) { return o->t[(size_t)layer * o->batch + b]; }
int oracle_n_obs(const corm_oracle *o, int layer, int b) { return o->n_obs[(size_t)layer * o->batch + b]; }

/* Copies the live entries of one unit, in order: k/v [live,d] doubles, word [live], pos [live]. */
int oracle_export_unit(const corm_oracle *o, int layer, int b, int h, double *k, double *v, uint32_t *word,
                       int *pos) {
    size_t u = unit_index(o, layer, b, h), C = (size_t)o->max_tokens, d = (size_t)o->head_dim;
    int l = o->live[u];
    if (k) memcpy(k, o->k + u * C * d, (size_t)l * d * sizeof(double));
    if (v) memcpy(v, o->v + u * C * d, (size_t)l * d * sizeof(double));
    if (word) for (int j = 0; j < l; ++j) word[j] = o->word[(u * C + j) * REG_WORDS];   /* newest 32 verdicts */
    if (pos) memcpy(pos, o->pos + u * C, (size_t)l * sizeof(int));
    return l;
}

/* Copies the whole registers of one unit's live entries, in order: regs [live][REG_WORDS], word 0 = newest 32
 * verdicts (bit b of the register = verdict of the query b steps ago, Algorithm 1's message column). */
int oracle_export_registers(const corm_oracle *o, int layer, int b, int h, uint32_t *regs) {
    size_t u = unit_index(o, layer, b, h), C = (size_t)o->max_tokens;
    int l = o->live[u];
    memcpy(regs, o->word + u * C * REG_WORDS, (size_t)l * REG_WORDS * sizeof(uint32_t));
    return l;
}

int oracle_register_words(void) { return REG_WORDS; }

/* Replaces one unit's entries and its sequence counters (used to start both sides from the same state, and as a
 * checkpoint restore). regs: [live][REG_WORDS] whole registers as oracle_export_registers gives them. */
int oracle_import_unit_full(corm_oracle *o, int layer, int b, int h, int live, const double *k, const double *v,
                            const uint32_t *regs, const int *pos, int n_tokens, int n_obs) {
    if (live < 0 || live > o->max_tokens) return ORACLE_CAPACITY;
    size_t u = unit_index(o, layer, b, h), C = (size_t)o->max_tokens, d = (size_t)o->head_dim;
    memcpy(o->k + u * C * d, k, (size_t)live * d * sizeof(double));
    memcpy(o->v + u * C * d, v, (size_t)live * d * sizeof(double));
    memcpy(o->word + u * C * REG_WORDS, regs, (size_t)live * REG_WORDS * sizeof(uint32_t));
    memcpy(o->pos + u * C, pos, (size_t)live * sizeof(int));
    o->live[u] = live;
    o->t[(size_t)layer * o->batch + b] = n_tokens;
    o->n_obs[(size_t)layer * o->batch + b] = n_obs;
    return ORACLE_OK;
}

/* The same with one 32-bit word per entry (the newest 32 verdicts): all of the register only for windows of up to
 * 32 queries, so wider windows are refused rather than silently losing verdicts. */
int oracle_import_unit(corm_oracle *o, int layer, int b, int h, int live, const double *k, const double *v,
                       const uint32_t *word, const int *pos, int n_tokens, int n_obs) {
    if (o->w > 32) return ORACLE_BAD_ARG;
    if (live < 0 || live > o->max_tokens) return ORACLE_CAPACITY;
    size_t u = unit_index(o, layer, b, h), C = (size_t)o->max_tokens, d = (size_t)o->head_dim;
    memcpy(o->k + u * C * d, k, (size_t)live * d * sizeof(double));
    memcpy(o->v + u * C * d, v, (size_t)live * d * sizeof(double));
    for (int j = 0; j < live; ++j) { reg_clear(o->word + (u * C + j) * REG_WORDS); o->word[(u * C + j) * REG_WORDS] = word[j]; }
    memcpy(o->pos + u * C, pos, (size_t)live * sizeof(int));
    o->live[u] = live;
    o->t[(size_t)layer * o->batch + b] = n_tokens;
    o->n_obs[(size_t)layer * o->batch + b] = n_obs;
    return ORACLE_OK;
}

/* For each live entry: how many queries ago it was last judged important (0 = by the latest query), -1 if by none
 * of the last w. This is all of the register that can still influence an eviction. */
int oracle_export_age(const corm_oracle *o, int layer, int b, int h, int *age) {
    size_t u = unit_index(o, layer, b, h), C = (size_t)o->max_tokens;
    int l = o->live[u];
    for (int j = 0; j < l; ++j) {
        const uint32_t *reg = o->word + (u * C + j) * REG_WORDS;
        age[j] = -1;
        for (int bit = 0; bit < o->w && age[j] < 0; ++bit)
            if ((reg[bit >> 5] >> (bit & 31)) & 1u) age[j] = bit;
    }
    return l;
}

void oracle_counters(const corm_oracle *o, long long *appended, long long *evicted, long long *verdict_evals,
                     long long *near_threshold) {
    if (appended) *appended = o->appended;
    if (evicted) *evicted = o->evicted;
    if (verdict_evals) *verdict_evals = o->verdict_evals;
    if (near_threshold) *near_threshold = o->near_threshold;
}

void oracle_set_near_band(corm_oracle *o, double rel) { o->near_rel = rel; }
