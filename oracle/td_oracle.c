/*
 * CPU oracle for the transfer dock (see td_oracle.h: test infrastructure only).
 * Plain C, one thread, no blocking or fusion: every function is the definition
 * written out, in the order the workflow of "Distributed Transfer Dock Strategy"
 * states it (metadata request -> data get/put -> state update).
 */
#include "td_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

#define ROW_ALIGN 8u   /* rows start on multiples of 8 elements inside an arena */

struct ora_dock {
    uint32_t G, N, S, n, ncol, ncons;
    ora_column   col[32];
    ora_consumer cons[32];
    uint64_t cap[3];            /* elements per shard, by length class (1, 2) */
    uint32_t reward_column;
    double   eps;
    uint32_t *status;           /* [n] bit c = column c stored                */
    int32_t  *len[3];           /* [n] per length class, -1 = unset           */
    int64_t  *off[3];           /* [n] element offset inside the shard arena  */
    uint64_t *cursor[3];        /* [S] next free element per shard            */
    uint8_t  *arena[32];        /* ragged column: S * cap * esize bytes       */
    uint8_t  *scalar[32];       /* scalar column: n * esize bytes             */
    uint32_t *claim[32];        /* per consumer, bit per group                */
    uint32_t *consumed[32];     /* per consumer, bit per sample               */
    ora_stats stats;
};

static size_t esize(int dtype) { return dtype == ORA_BF16 ? 2 : 4; }
static uint64_t align_up(uint64_t x) { return (x + ROW_ALIGN - 1) / ROW_ALIGN * ROW_ALIGN; }

/* Warehouses split the batch along the prompt dimension: contiguous blocks of
 * whole prompts, so a group never straddles two shards. */
uint32_t ora_shard_of(const ora_dock *d, uint32_t s) {
    uint32_t prompt = s / d->N;
    return prompt / (d->G / d->S);
}

static int get_bit(const uint32_t *w, uint32_t i) { return (w[i >> 5] >> (i & 31)) & 1u; }
static void set_bit(uint32_t *w, uint32_t i) { w[i >> 5] |= 1u << (i & 31); }

ora_dock *ora_create(const ora_config *cfg) {
    if (!cfg || cfg->n_columns == 0 || cfg->n_columns > 32 || cfg->n_consumers == 0 ||
        cfg->n_consumers > 32 || cfg->n_prompts == 0 || cfg->n_per_group == 0 ||
        cfg->n_shards == 0 || cfg->n_prompts % cfg->n_shards != 0)
        return NULL;
    for (uint32_t k = 0; k < cfg->n_consumers; ++k) {
        const ora_consumer *K = &cfg->consumers[k];
        if (K->out_mask & ~K->need_mask) return NULL;          /* only ready columns are served */
        if ((K->flags & ORA_F_ADVANTAGE) &&
            (cfg->reward_column >= cfg->n_columns || !((K->need_mask >> cfg->reward_column) & 1u) ||
             cfg->columns[cfg->reward_column].cls != ORA_SCALAR ||
             cfg->columns[cfg->reward_column].dtype != ORA_F32))
            return NULL;
    }
    ora_dock *d = (ora_dock *)calloc(1, sizeof(*d));
    d->G = cfg->n_prompts; d->N = cfg->n_per_group; d->S = cfg->n_shards;
    d->n = d->G * d->N; d->ncol = cfg->n_columns; d->ncons = cfg->n_consumers;
    d->cap[ORA_PROMPT] = align_up(cfg->prompt_elems_per_shard);
    d->cap[ORA_RESPONSE] = align_up(cfg->response_elems_per_shard);
    d->reward_column = cfg->reward_column;
    d->eps = (double)cfg->adv_eps;
    memcpy(d->col, cfg->columns, d->ncol * sizeof(ora_column));
    memcpy(d->cons, cfg->consumers, d->ncons * sizeof(ora_consumer));
    d->status = (uint32_t *)calloc(d->n, sizeof(uint32_t));
    for (int L = 1; L <= 2; ++L) {
        d->len[L] = (int32_t *)malloc(d->n * sizeof(int32_t));
        d->off[L] = (int64_t *)malloc(d->n * sizeof(int64_t));
        d->cursor[L] = (uint64_t *)calloc(d->S, sizeof(uint64_t));
    }
    for (uint32_t c = 0; c < d->ncol; ++c) {
        if (d->col[c].cls == ORA_SCALAR)
            d->scalar[c] = (uint8_t *)calloc(d->n, esize(d->col[c].dtype));
        else
            d->arena[c] = (uint8_t *)calloc((size_t)d->S * d->cap[d->col[c].cls] + 1,
                                            esize(d->col[c].dtype));
    }
    for (uint32_t k = 0; k < d->ncons; ++k) {
        d->claim[k] = (uint32_t *)calloc((d->G + 31) / 32, sizeof(uint32_t));
        d->consumed[k] = (uint32_t *)calloc((d->n + 31) / 32, sizeof(uint32_t));
    }
    ora_reset(d);
    return d;
}

void ora_destroy(ora_dock *d) {
    if (!d) return;
    free(d->status);
    for (int L = 1; L <= 2; ++L) { free(d->len[L]); free(d->off[L]); free(d->cursor[L]); }
    for (uint32_t c = 0; c < 32; ++c) { free(d->arena[c]); free(d->scalar[c]); }
    for (uint32_t k = 0; k < 32; ++k) { free(d->claim[k]); free(d->consumed[k]); }
    free(d);
}

/* One buffer serves one RL iteration; a reset forgets every table and bitmap
 * but leaves payload bytes and capacities alone. */
void ora_reset(ora_dock *d) {
    memset(d->status, 0, d->n * sizeof(uint32_t));
    for (int L = 1; L <= 2; ++L) {
        for (uint32_t s = 0; s < d->n; ++s) { d->len[L][s] = -1; d->off[L][s] = -1; }
        memset(d->cursor[L], 0, d->S * sizeof(uint64_t));
    }
    for (uint32_t k = 0; k < d->ncons; ++k) {
        memset(d->claim[k], 0, (d->G + 31) / 32 * sizeof(uint32_t));
        memset(d->consumed[k], 0, (d->n + 31) / 32 * sizeof(uint32_t));
    }
    memset(&d->stats, 0, sizeof(d->stats));
}

static void flag(ora_dock *d, uint32_t bit, uint64_t *counter) {
    d->stats.error_word |= bit;
    ++*counter;
}

/*
 * Workflow step 2 (a worker sends real data to the warehouses) followed by step 3
 * (the warehouse updates its state, which every controller sees).  Samples are
 * taken one by one in call order.  Reading for what the paper leaves open:
 *   - a row's place is fixed by the first column of its length class to arrive:
 *     the next free element of its shard, rows starting on multiples of 8 elements;
 *   - a second put of the same (sample, column) is dropped, the first one stays;
 *   - a later column of the same class must bring the same length.
 */
int64_t ora_put(ora_dock *d, uint32_t column, const int32_t *indices, uint32_t k,
                const int32_t *cu, const void *data) {
    if (!d || column >= d->ncol || (k && !indices) || (k && !data)) return -1;
    const ora_column *C = &d->col[column];
    const size_t es = esize(C->dtype);
    const uint32_t bit = 1u << column;
    if (C->cls != ORA_SCALAR && k && !cu) return -1;
    int64_t accepted = 0;
    for (uint32_t i = 0; i < k; ++i) {
        int32_t s = indices[i];
        if (s < 0 || (uint32_t)s >= d->n) { flag(d, ORA_ERR_OOB_INDEX, &d->stats.n_oob); continue; }
        if (d->status[s] & bit) { flag(d, ORA_ERR_DUP_PUT, &d->stats.n_dup); continue; }
        if (C->cls == ORA_SCALAR) {
            memcpy(d->scalar[column] + (size_t)s * es, (const uint8_t *)data + (size_t)i * es, es);
        } else {
            const int L = C->cls;
            int64_t l = (int64_t)cu[i + 1] - (int64_t)cu[i];
            if (l < 0) { flag(d, ORA_ERR_BAD_LENGTH, &d->stats.n_bad_length); continue; }
            uint32_t sh = ora_shard_of(d, (uint32_t)s);
            if (d->len[L][s] < 0) {
                uint64_t need = align_up((uint64_t)l);
                if (d->cursor[L][sh] + need > d->cap[L]) {
                    flag(d, ORA_ERR_ARENA_FULL, &d->stats.n_arena_full);
                    continue;
                }
                d->len[L][s] = (int32_t)l;
                d->off[L][s] = (int64_t)d->cursor[L][sh];
                d->cursor[L][sh] += need;
            } else if (d->len[L][s] != l) {
                flag(d, ORA_ERR_LEN_MISMATCH, &d->stats.n_len_mismatch);
                continue;
            }
            uint8_t *dst = d->arena[column] + ((size_t)sh * d->cap[L] + (size_t)d->off[L][s]) * es;
            memcpy(dst, (const uint8_t *)data + (size_t)cu[i] * es, (size_t)l * es);
        }
        d->status[s] |= bit;
        ++accepted;
    }
    d->stats.put_accepted[column] += (uint64_t)accepted;
    return accepted;
}

static int wanted(const ora_dock *d, const ora_consumer *K, const ora_get_out *out, uint32_t c) {
    return c < d->ncol && ((K->out_mask >> c) & 1u) && out->col[c] != NULL;
}

/* The fused stream joins a prompt-length and a response-length column of one element size, both
 * among the consumer's output columns; its advantage twin needs the advantages. */
static int seq_args_ok(const ora_dock *d, const ora_consumer *K, const ora_get_out *out) {
    if (out->seq) {
        uint32_t cp = out->seq_prompt_col, cr = out->seq_response_col;
        if (cp >= d->ncol || cr >= d->ncol) return 0;
        if (d->col[cp].cls != ORA_PROMPT || d->col[cr].cls != ORA_RESPONSE) return 0;
        if (esize(d->col[cp].dtype) != esize(d->col[cr].dtype)) return 0;
        if (!((K->out_mask >> cp) & 1u) || !((K->out_mask >> cr) & 1u)) return 0;
    }
    if (out->seq_advantages && !((K->flags & ORA_F_ADVANTAGE) && out->advantages)) return 0;
    return 1;
}

/* Would `count` samples with these token totals and this longest row still fit
 * every buffer the caller supplied? */
static int fits(const ora_dock *d, const ora_consumer *K, const ora_get_out *out,
                uint64_t count, uint64_t tokP, uint64_t tokR, uint32_t maxP, uint32_t maxR) {
    for (uint32_t c = 0; c < d->ncol; ++c) {
        if (!wanted(d, K, out, c)) continue;
        uint64_t cap = out->col_capacity_elems[c];
        int cls = d->col[c].cls;
        if (cls == ORA_SCALAR) {
            if (count > cap) return 0;
        } else if (out->mode == ORA_PACKED) {
            if ((cls == ORA_PROMPT ? tokP : tokR) > cap) return 0;
        } else {
            uint32_t W = cls == ORA_PROMPT ? out->pad_prompt_to : out->pad_response_to;
            uint32_t longest = cls == ORA_PROMPT ? maxP : maxR;
            if (longest > W || count * (uint64_t)W > cap) return 0;
        }
    }
    if ((out->seq || out->seq_advantages) && tokP + tokR > out->seq_capacity_elems) return 0;
    return 1;
}

/* Steps "obtain real data from distributed storage" for a fixed list of samples:
 * cu_seqlens, the gathered columns and the group-normalised advantage. */
static void emit(const ora_dock *d, const ora_consumer *K, const int32_t *idx, uint32_t count,
                 const ora_get_out *out, uint64_t *tokP, uint64_t *tokR) {
    const int32_t *lenP = d->len[ORA_PROMPT], *lenR = d->len[ORA_RESPONSE];
    /* cu_seqlens: prefix sums of the true lengths, leading zero */
    int64_t p = 0, r = 0;
    if (out->cu_prompt) out->cu_prompt[0] = 0;
    if (out->cu_response) out->cu_response[0] = 0;
    if (out->cu_seq) out->cu_seq[0] = 0;
    for (uint32_t i = 0; i < count; ++i) {
        int32_t s = idx[i];
        p += lenP[s] > 0 ? lenP[s] : 0;
        r += lenR[s] > 0 ? lenR[s] : 0;
        if (out->cu_prompt) out->cu_prompt[i + 1] = (int32_t)p;
        if (out->cu_response) out->cu_response[i + 1] = (int32_t)r;
        if (out->cu_seq) out->cu_seq[i + 1] = (int32_t)(p + r);
    }
    *tokP = (uint64_t)p; *tokR = (uint64_t)r;
    /* columns */
    for (uint32_t c = 0; c < d->ncol; ++c) {
        if (!wanted(d, K, out, c)) continue;
        const ora_column *C = &d->col[c];
        const size_t es = esize(C->dtype);
        uint8_t *dst = (uint8_t *)out->col[c];
        if (C->cls == ORA_SCALAR) {
            for (uint32_t i = 0; i < count; ++i)
                memcpy(dst + (size_t)i * es, d->scalar[c] + (size_t)idx[i] * es, es);
            continue;
        }
        const int L = C->cls;
        const uint32_t W = L == ORA_PROMPT ? out->pad_prompt_to : out->pad_response_to;
        size_t at = 0;   /* packed write position, elements */
        for (uint32_t i = 0; i < count; ++i) {
            int32_t s = idx[i];
            size_t l = d->len[L][s] > 0 ? (size_t)d->len[L][s] : 0;
            const uint8_t *src = d->arena[c] +
                ((size_t)ora_shard_of(d, (uint32_t)s) * d->cap[L] + (size_t)(d->off[L][s] > 0 ? d->off[L][s] : 0)) * es;
            if (out->mode == ORA_PACKED) {
                memcpy(dst + at * es, src, l * es);
                at += l;
            } else {
                /* a row of W elements: the l stored ones and W - l copies of the pad pattern,
                 * behind them, or in front of them for a prompt that is asked for left-padded */
                uint8_t *row = dst + (size_t)i * W * es;
                const size_t lead = (L == ORA_PROMPT && (out->flags & ORA_OUT_LEFT_PAD_PROMPT)) ? W - l : 0;
                for (size_t j = 0; j < lead; ++j) memcpy(row + j * es, &C->pad_bits, es);
                memcpy(row + lead * es, src, l * es);
                for (size_t j = lead + l; j < W; ++j) memcpy(row + j * es, &C->pad_bits, es);
            }
        }
    }
    /* Group-normalised advantage, per group of N consecutive samples, in double:
     * A = (r - mean) / (std + eps) with the population standard deviation. */
    if ((K->flags & ORA_F_ADVANTAGE) && out->advantages) {
        const float *rew = (const float *)d->scalar[d->reward_column];
        for (uint32_t g0 = 0; g0 + d->N <= count; g0 += d->N) {
            double sum = 0.0;
            for (uint32_t j = 0; j < d->N; ++j) sum += (double)rew[idx[g0 + j]];
            double mean = sum / (double)d->N;
            double ss = 0.0;
            for (uint32_t j = 0; j < d->N; ++j) {
                double dv = (double)rew[idx[g0 + j]] - mean;
                ss += dv * dv;
            }
            double sd = sqrt(ss / (double)d->N);
            for (uint32_t j = 0; j < d->N; ++j)
                out->advantages[g0 + j] = (float)(((double)rew[idx[g0 + j]] - mean) / (sd + d->eps));
        }
    }
    /* Fused stream: what a varlen trainer reads directly.  Sample i occupies elements
     * [cu_seq[i], cu_seq[i+1]): its prompt row, then its response row. */
    if (out->seq || out->seq_advantages) {
        const uint32_t cp = out->seq_prompt_col, cr = out->seq_response_col;
        const size_t es = out->seq ? esize(d->col[cp].dtype) : 0;
        size_t at = 0;
        for (uint32_t i = 0; i < count; ++i) {
            int32_t s = idx[i];
            size_t lp = lenP[s] > 0 ? (size_t)lenP[s] : 0, lr = lenR[s] > 0 ? (size_t)lenR[s] : 0;
            size_t sh = ora_shard_of(d, (uint32_t)s);
            if (out->seq) {
                const uint8_t *srcP = d->arena[cp] +
                    (sh * d->cap[ORA_PROMPT] + (size_t)(d->off[ORA_PROMPT][s] > 0 ? d->off[ORA_PROMPT][s] : 0)) * es;
                const uint8_t *srcR = d->arena[cr] +
                    (sh * d->cap[ORA_RESPONSE] + (size_t)(d->off[ORA_RESPONSE][s] > 0 ? d->off[ORA_RESPONSE][s] : 0)) * es;
                memcpy((uint8_t *)out->seq + at * es, srcP, lp * es);
                memcpy((uint8_t *)out->seq + (at + lp) * es, srcR, lr * es);
            }
            if (out->seq_advantages) {
                for (size_t j = 0; j < lp; ++j) out->seq_advantages[at + j] = 0.0f;
                for (size_t j = 0; j < lr; ++j) out->seq_advantages[at + lp + j] = out->advantages[i];
            }
            at += lp + lr;
        }
    }
}

/*
 * Workflow step 1 (the worker state asks its controller which samples come next)
 * and step 2 (it fetches them).  Reading: lowest group index first, whole GRPO
 * groups only, a group is served to a consumer once; fewer ready groups than
 * asked for is not an error.  The scan stops before the first group that would
 * not fit a supplied buffer; that group stays unclaimed.
 */
int ora_get(ora_dock *d, uint32_t consumer, uint32_t max_samples, const ora_get_out *out) {
    if (!d || !out || consumer >= d->ncons || !out->indices || !out->result) return -1;
    if (out->flags & ~(uint32_t)ORA_OUT_LEFT_PAD_PROMPT) return -1;
    const uint32_t m = max_samples / d->N;
    if (m == 0) return -1;
    ora_consumer *K = &d->cons[consumer];
    if (!seq_args_ok(d, K, out)) return -1;
    uint32_t taken = 0, status = 0;
    uint64_t tokP = 0, tokR = 0;
    uint32_t maxP = 0, maxR = 0;
    for (uint32_t g = 0; g < d->G && taken < m; ++g) {
        if (get_bit(d->claim[consumer], g)) continue;
        int ready = 1;
        for (uint32_t j = 0; j < d->N; ++j)
            if ((d->status[g * d->N + j] & K->need_mask) != K->need_mask) { ready = 0; break; }
        if (!ready) continue;
        uint64_t gP = 0, gR = 0; uint32_t mP = maxP, mR = maxR;
        for (uint32_t j = 0; j < d->N; ++j) {
            uint32_t s = g * d->N + j;
            uint32_t lp = d->len[ORA_PROMPT][s] > 0 ? (uint32_t)d->len[ORA_PROMPT][s] : 0;
            uint32_t lr = d->len[ORA_RESPONSE][s] > 0 ? (uint32_t)d->len[ORA_RESPONSE][s] : 0;
            gP += lp; gR += lr;
            if (lp > mP) mP = lp;
            if (lr > mR) mR = lr;
        }
        if (!fits(d, K, out, (uint64_t)(taken + 1) * d->N, tokP + gP, tokR + gR, mP, mR)) {
            status |= ORA_ERR_OUT_TRUNC;
            flag(d, ORA_ERR_OUT_TRUNC, &d->stats.n_truncated);
            break;
        }
        set_bit(d->claim[consumer], g);
        for (uint32_t j = 0; j < d->N; ++j) {
            set_bit(d->consumed[consumer], g * d->N + j);
            out->indices[taken * d->N + j] = (int32_t)(g * d->N + j);
        }
        tokP += gP; tokR += gR; maxP = mP; maxR = mR;
        ++taken;
    }
    uint64_t eP, eR;
    emit(d, K, out->indices, taken * d->N, out, &eP, &eR);
    out->result->n_samples = taken * d->N;
    out->result->n_groups = taken;
    out->result->prompt_tokens = eP;
    out->result->response_tokens = eR;
    out->result->status = status;
    d->stats.got_samples[consumer] += (uint64_t)taken * d->N;
    d->stats.got_tokens[consumer] += eP + eR;
    return 0;
}

int ora_gather(const ora_dock *d, uint32_t consumer, const int32_t *indices, uint32_t count,
               const ora_get_out *out) {
    if (!d || !out || consumer >= d->ncons || (count && !indices)) return -1;
    if (out->flags & ~(uint32_t)ORA_OUT_LEFT_PAD_PROMPT) return -1;
    const ora_consumer *K = &d->cons[consumer];
    if (!seq_args_ok(d, K, out)) return -1;
    uint64_t tokP = 0, tokR = 0; uint32_t maxP = 0, maxR = 0;
    for (uint32_t i = 0; i < count; ++i) {
        int32_t s = indices[i];
        if (s < 0 || (uint32_t)s >= d->n) return -1;
        uint32_t lp = d->len[ORA_PROMPT][s] > 0 ? (uint32_t)d->len[ORA_PROMPT][s] : 0;
        uint32_t lr = d->len[ORA_RESPONSE][s] > 0 ? (uint32_t)d->len[ORA_RESPONSE][s] : 0;
        tokP += lp; tokR += lr;
        if (lp > maxP) maxP = lp;
        if (lr > maxR) maxR = lr;
    }
    if (!fits(d, K, out, count, tokP, tokR, maxP, maxR)) return -1;
    if (out->indices && out->indices != indices)
        memcpy(out->indices, indices, count * sizeof(int32_t));
    uint64_t eP, eR;
    emit(d, K, indices, count, out, &eP, &eR);
    if (out->result) {
        out->result->n_samples = count;
        out->result->n_groups = count / d->N;
        out->result->prompt_tokens = eP;
        out->result->response_tokens = eR;
        out->result->status = 0;
    }
    return 0;
}

void ora_get_stats(const ora_dock *d, ora_stats *out) { *out = d->stats; }
const uint32_t *ora_status(const ora_dock *d) { return d->status; }
const int32_t  *ora_len(const ora_dock *d, int cls) { return d->len[cls]; }
const int64_t  *ora_off(const ora_dock *d, int cls) { return d->off[cls]; }
const uint64_t *ora_cursor(const ora_dock *d, int cls) { return d->cursor[cls]; }
const uint32_t *ora_claim(const ora_dock *d, uint32_t k) { return d->claim[k]; }
const uint32_t *ora_consumed(const ora_dock *d, uint32_t k) { return d->consumed[k]; }
const void *ora_arena(const ora_dock *d, uint32_t c, uint32_t sh) {
    if (!d->arena[c]) return NULL;
    return d->arena[c] + (size_t)sh * d->cap[d->col[c].cls] * esize(d->col[c].dtype);
}
const void *ora_scalars(const ora_dock *d, uint32_t c) { return d->scalar[c]; }

/* Eq. 1: what one actor-update request moves out of a centralized buffer. */
double ora_cv(double G, double N, double B, double PL, double n, double SL, double M) {
    return G * N * B * (PL + n * SL + M) / (1024.0 * 1024.0 * 1024.0);
}
/* Eq. 2: total over the last three steps of the replay-buffer workflow. */
double ora_tcv(double G, double N, double B, double PL, double n, double SL, double M) {
    return G * N * B * (2.0 * PL + 3.0 * n * SL + 8.0 * M) / (1024.0 * 1024.0 * 1024.0);
}
/* Eq. 4: per-warehouse share with C controllers and S warehouses. */
double ora_tcv_dock(double G, double N, double B, double PL, double n, double SL, double M,
                    double C, double S) {
    return G * N * B * (2.0 * PL + 3.0 * n * SL + 8.0 * (C + 1.0) * M) / S / (1024.0 * 1024.0 * 1024.0);
}
