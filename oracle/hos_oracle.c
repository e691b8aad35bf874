/*
 * CPU oracle for the hybrid offline-online scheduler (arXiv 2502.15763).
 * TEST INFRASTRUCTURE ONLY -- see hos_oracle.h.  Single thread, no blocking,
 * no fusion: each function takes the steps of the definition in order.
 */
#include "hos_oracle.h"

#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------- */
/* Offline part: Minimizing-Makespan Bin Packing, Eq. 26-30                   */
/* ------------------------------------------------------------------------- */

void ora_estimate(int n, const uint32_t* p, const uint32_t* o, const ora_cost* c, int64_t* T)
{
    for (int i = 0; i < n; ++i)
        T[i] = (int64_t)c->est_per_prompt_token * (int64_t)p[i]
             + (int64_t)c->est_per_output_token * (int64_t)o[i];
}

typedef struct { int64_t key; int32_t idx; } ora_keyed;

/* larger key first; equal keys: smaller index first */
static int cmp_key_desc_idx_asc(const void* a, const void* b)
{
    const ora_keyed* x = (const ora_keyed*)a;
    const ora_keyed* y = (const ora_keyed*)b;
    if (x->key != y->key) return (x->key > y->key) ? -1 : 1;
    if (x->idx != y->idx) return (x->idx < y->idx) ? -1 : 1;
    return 0;
}

void ora_order(int n, const int64_t* T, int32_t* order)
{
    ora_keyed* a = (ora_keyed*)malloc(sizeof(ora_keyed) * (size_t)(n > 0 ? n : 1));
    for (int i = 0; i < n; ++i) { a[i].key = T[i]; a[i].idx = i; }
    qsort(a, (size_t)n, sizeof(ora_keyed), cmp_key_desc_idx_asc);   /* keys (T, i) are unique */
    for (int r = 0; r < n; ++r) order[r] = a[r].idx;
    free(a);
}

void ora_lpt(int n, int M, const int64_t* T, const int32_t* order, int32_t* assign, int64_t* load)
{
    for (int j = 0; j < M; ++j) load[j] = 0;
    for (int r = 0; r < n; ++r) {
        int i = order[r];
        int best = 0;                               /* smallest j attaining the minimum load */
        for (int j = 1; j < M; ++j)
            if (load[j] < load[best]) best = j;
        assign[i] = best;
        load[best] += T[i];
    }
}

/* One round: enumerate EVERY candidate (i, k, u) and keep the lexicographic minimum of
 * (v, i, k, u), u = -1 meaning "move".  Returns 1 and applies it when v < Lmax. */
static int local_search_round(int n, int M, const int64_t* T, int32_t* assign, int64_t* load,
                              ora_move* out)
{
    int jmax = 0;                                   /* smallest j attaining the maximum load */
    for (int j = 1; j < M; ++j)
        if (load[j] > load[jmax]) jmax = j;
    const int64_t Lmax = load[jmax];

    int have = 0;
    int64_t bv = 0; int bi = -1, bk = -1, bu = -1;

    for (int i = 0; i < n; ++i) {
        if (assign[i] != jmax) continue;
        /* u = -1 .. n-1; u = -1 stands for "move i", tried once for every other client k;
         * u >= 0 is a swap with request u, whose client fixes k; needs d = T_i - T_u > 0 */
        for (int u = -1; u < n; ++u) {
            int k_first, k_last;
            if (u < 0) { k_first = 0; k_last = M - 1; }
            else {
                if (assign[u] == jmax) continue;
                k_first = k_last = assign[u];
            }
            for (int k = k_first; k <= k_last; ++k) {
                if (k == jmax) continue;
                int64_t d = (u < 0) ? T[i] : T[i] - T[u];
                if (u >= 0 && d <= 0) continue;
                int64_t a = Lmax - d, b = load[k] + d;
                int64_t v = (a > b) ? a : b;
                int better;
                if (!have) better = 1;
                else if (v != bv) better = v < bv;
                else if (i != bi) better = i < bi;
                else if (k != bk) better = k < bk;
                else better = u < bu;
                if (better) { have = 1; bv = v; bi = i; bk = k; bu = u; }
            }
        }
    }
    if (!have || bv >= Lmax) {
        out->i = -1; out->u = -1; out->k = -1; out->v = Lmax;
        return 0;
    }
    int64_t d = (bu < 0) ? T[bi] : T[bi] - T[bu];
    assign[bi] = bk;
    if (bu >= 0) assign[bu] = jmax;
    load[jmax] -= d;
    load[bk]   += d;
    out->i = bi; out->u = bu; out->k = bk; out->v = bv;
    return 1;
}

int ora_local_search(int n, int M, const int64_t* T, int32_t* assign, int64_t* load,
                     int rounds, ora_move* log)
{
    int applied = 0;
    for (int r = 0; r < rounds; ++r) {
        ora_move mv;
        int ok = local_search_round(n, M, T, assign, load, &mv);
        if (log) log[r] = mv;
        if (ok) { ++applied; continue; }
        /* a no-op round leaves the state unchanged, so every later round is the same no-op */
        if (log) for (int s = r + 1; s < rounds; ++s) log[s] = mv;
        break;
    }
    return applied;
}

/* ------------------------------------------------------------------------- */
/* A stronger packing for Eq. 26-30: MULTIFIT (Coffman, Garey and Johnson,    */
/* "An application of bin-packing to multiprocessor scheduling", 1978)        */
/* ------------------------------------------------------------------------- */

/* First-fit decreasing with capacity C: every request, longest first, goes to the LOWEST client
 * on which it still fits (load + T <= C).  Returns 1 when every request found a client. */
static int first_fit_decreasing(int n, int M, const int64_t* T, const int32_t* order, int64_t C,
                                int32_t* assign, int64_t* load)
{
    for (int j = 0; j < M; ++j) load[j] = 0;
    for (int r = 0; r < n; ++r) {
        int i = order[r];
        int j = 0;
        while (j < M && load[j] + T[i] > C) ++j;
        if (j == M) return 0;
        assign[i] = j;
        load[j] += T[i];
    }
    return 1;
}

/* MULTIFIT: bisection on the capacity.  The search starts from the interval the authors give,
 * C_L = max(ceil(sum T / M), max T) (no packing can do better) and C_U = max(ceil(2 sum T / M), max T)
 * (first-fit decreasing always succeeds there), in integers: while C_L < C_U and steps remain,
 * C = floor((C_L + C_U) / 2); success -> C_U = C, failure -> C_L = C + 1.  The packing is the
 * first-fit decreasing one at the final C_U.  Returns 1 and fills assign/load when that packing
 * exists (always, by the authors' result on C_U), 0 otherwise; *C_final gets the capacity. */
int ora_multifit(int n, int M, const int64_t* T, const int32_t* order, int max_steps,
                 int32_t* assign, int64_t* load, int64_t* C_final)
{
    int64_t sumT = 0, maxT = 0;
    for (int i = 0; i < n; ++i) { sumT += T[i]; if (T[i] > maxT) maxT = T[i]; }
    int64_t lo = (sumT + M - 1) / M;
    if (maxT > lo) lo = maxT;
    int64_t hi = (2 * sumT + M - 1) / M;
    if (maxT > hi) hi = maxT;
    for (int step = 0; step < max_steps && lo < hi; ++step) {
        int64_t C = lo + (hi - lo) / 2;
        if (first_fit_decreasing(n, M, T, order, C, assign, load)) hi = C;
        else lo = C + 1;
    }
    if (C_final) *C_final = hi;
    return first_fit_decreasing(n, M, T, order, hi, assign, load);
}

/* The optimum of Eq. 26-30 by trying every assignment (M^n of them): for tiny instances only. */
static void optimum_rec(int n, int M, const int64_t* T, int i, int64_t* load, int64_t* best)
{
    if (i == n) {
        int64_t m = 0;
        for (int j = 0; j < M; ++j) if (load[j] > m) m = load[j];
        if (*best < 0 || m < *best) *best = m;
        return;
    }
    for (int j = 0; j < M; ++j) {
        load[j] += T[i];
        optimum_rec(n, M, T, i + 1, load, best);
        load[j] -= T[i];
    }
}

int64_t ora_optimal_makespan(int n, int M, const int64_t* T)
{
    int64_t* load = (int64_t*)calloc((size_t)M, sizeof(int64_t));
    int64_t best = -1;
    optimum_rec(n, M, T, 0, load, &best);
    free(load);
    return best < 0 ? 0 : best;
}

/* ------------------------------------------------------------------------- */
/* Lower bounds, Eq. 31-32                                                    */
/* ------------------------------------------------------------------------- */

static int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

/* Duration of a prefill stage over `tokens` prompt tokens: affine, or by level (Eq. 5-7). */
static int64_t prefill_us(const ora_cost* c, int64_t tokens)
{
    if (c->n_levels == 0)
        return (int64_t)c->prefill_fixed_us + (int64_t)c->prefill_per_token_us * tokens;
    for (uint32_t l = 0; l < c->n_levels; ++l)
        if (tokens <= (int64_t)c->level_cap[l]) return (int64_t)c->level_time[l];
    return (int64_t)c->level_time[c->n_levels - 1];        /* not reached: admission stops at the largest level */
}

/* Does a prefill stage that already holds `have` tokens take `more` on top?  (largest level's capacity) */
static int stage_holds(const ora_cost* c, int64_t have, int64_t more)
{
    return c->n_levels == 0 || have + more <= (int64_t)c->level_cap[c->n_levels - 1];
}

void ora_lower_bound(int n, int M, int cap, const uint32_t* p, const uint32_t* o,
                     const ora_cost* c, ora_lb* out)
{
    const int64_t ad = c->decode_fixed_us,  bd = c->decode_per_seq_us, q = c->decode_kv_div;

    /* --- packing bound: the optimum of Eq. 26 is at least the mean load, the largest
     *     item, and the two smallest of the M+1 largest items together --- */
    int64_t* T = (int64_t*)malloc(sizeof(int64_t) * (size_t)(n > 0 ? n : 1));
    int32_t* order = (int32_t*)malloc(sizeof(int32_t) * (size_t)(n > 0 ? n : 1));
    ora_estimate(n, p, o, c, T);
    ora_order(n, T, order);
    int64_t sumT = 0, maxT = 0;
    for (int i = 0; i < n; ++i) { sumT += T[i]; if (T[i] > maxT) maxT = T[i]; }
    int64_t pairT = (n > M) ? T[order[M - 1]] + T[order[M]] : 0;
    int64_t lb = ceil_div(sumT, M);
    if (maxT > lb) lb = maxT;
    if (pairT > lb) lb = pairT;
    out->lb_pack = lb; out->sum_T = sumT; out->max_T = maxT; out->pair_T = pairT;

    /* --- simulation bound T^LB = t^p* + t^d*: prefill work and decode work taken as two
     *     separate groups, each with the fewest possible iterations --- */
    int64_t P = 0, O = 0, K = 0, chain = 0;
    for (int i = 0; i < n; ++i) {
        P += p[i];
        O += o[i];
        int64_t alone = prefill_us(c, p[i]);        /* request i served alone on a client */
        for (int64_t s = 0; s < (int64_t)o[i]; ++s) {
            K += (int64_t)p[i] + s;                 /* KV tokens attended by decode step s */
            alone += ad + bd + ((int64_t)p[i] + s) / q;
        }
        if (alone > chain) chain = alone;
    }
    int64_t tp_star, tp_paper = 0;
    if (c->n_levels == 0) {
        /* every prefill iteration admits at most cap prompts and pays a_p once */
        tp_star = (int64_t)c->prefill_fixed_us * ceil_div(n, cap) + (int64_t)c->prefill_per_token_us * P;
    } else {
        /* by level: at least ceil(n/cap) stages of at least the smallest level's time; and a stage
         * of level l carries at most N^cap_l tokens, so the P tokens cost at least
         * min_l floor(P / N^cap_l) T^p_l.  Eq. 31 as printed takes l = L only. */
        int64_t by_count = (int64_t)c->level_time[0] * ceil_div(n, cap);
        int64_t by_tokens = -1;
        for (uint32_t l = 0; l < c->n_levels; ++l) {
            int64_t v = (P / (int64_t)c->level_cap[l]) * (int64_t)c->level_time[l];
            if (by_tokens < 0 || v < by_tokens) by_tokens = v;
        }
        tp_star = by_count > by_tokens ? by_count : by_tokens;
        tp_paper = (P / (int64_t)c->level_cap[c->n_levels - 1]) * (int64_t)c->level_time[c->n_levels - 1];
    }
    out->tp_paper_us = tp_paper;
    /* every decode iteration advances at most cap requests; floor(S/q) > S/q - 1 */
    int64_t td_q = q * ((ad - 1) * ceil_div(O, cap) + bd * O) + K;      /* q * t^d*  */
    int64_t work = ceil_div(q * tp_star + td_q, q * (int64_t)M);        /* mean client time */
    out->tp_star_us = ceil_div(tp_star, M);
    out->td_star_us = ceil_div(td_q, q * (int64_t)M);
    out->chain_us   = chain;
    out->lb_sim_us  = (work > chain) ? work : chain;
    free(T); free(order);
}

/* ------------------------------------------------------------------------- */
/* Online part: Algorithm 1 (queue order) and the iteration simulator         */
/* ------------------------------------------------------------------------- */

void ora_queue_build(int n, int M, const int32_t* assign, const uint32_t* p, const uint32_t* o,
                     int mode, int32_t* q_off, int32_t* q_req)
{
    int pos = 0;
    ora_keyed* a = (ora_keyed*)malloc(sizeof(ora_keyed) * (size_t)(n > 0 ? n : 1));
    for (int j = 0; j < M; ++j) {
        q_off[j] = pos;
        int m = 0;
        for (int i = 0; i < n; ++i)
            if (assign[i] == j) {
                /* SORTED: longest N^p + N^d first; FCFS: arrival (index) order */
                a[m].key = (mode == ORA_QUEUE_SORTED) ? (int64_t)p[i] + (int64_t)o[i] : 0;
                a[m].idx = i;
                ++m;
            }
        qsort(a, (size_t)m, sizeof(ora_keyed), cmp_key_desc_idx_asc);
        for (int r = 0; r < m; ++r) q_req[pos++] = a[r].idx;
    }
    q_off[M] = pos;
    free(a);
}

/* Trace hash (a definition made for this checker and the library; the paper has none): h <- (h + dur + C1 kind_n +
 * C2 tokens + C3 aux) * M  mod 2^64 per record, in trace order, from h = INIT. */
#define ORA_HASH_INIT  0xCBF29CE484222325ull
#define ORA_HASH_C1    0x9E3779B1ull
#define ORA_HASH_C2    0x85EBCA77ull
#define ORA_HASH_C3    0xC2B2AE3Dull
#define ORA_HASH_M     0x27D4EB2Full

typedef struct { int64_t kv, rem, total; } ora_running;

/* kv_reserve > 0: every request reserves exactly that many KV tokens from admission to
 * retirement (the paper's experiment reserves the maximum input + output, five blocks, for each
 * request, because the output length is not known when it is admitted); 0: it reserves p + o. */
void ora_simulate_client(int qn, const int32_t* q_req, const uint32_t* p, const uint32_t* o,
                         const ora_cost* c, int cap, int64_t kv_budget, int64_t kv_reserve,
                         uint32_t lambda_q16,
                         uint32_t max_iters, ora_client* res, ora_rec* trace, int64_t trace_cap)
{
    const int64_t ad = c->decode_fixed_us,  bd = c->decode_per_seq_us, q = c->decode_kv_div;

    ora_running* R = (ora_running*)malloc(sizeof(ora_running) * (size_t)(cap > 0 ? cap : 1));
    int nR = 0;                 /* |R| */
    int head = 0;               /* next queue position */
    int64_t reserved = 0;       /* sum over R of the reservations */
    int64_t t = 0, busy = 0, Cd = 0;
    uint64_t hash = ORA_HASH_INIT;
    uint32_t n_pre = 0, n_dec = 0;
    uint64_t iters = 0;
    int32_t status = 0;

    while (nR > 0 || head < qn) {
        /* 1. candidates: a prefix of the queue, no skipping */
        int nA = 0; int64_t sumP = 0, sumTot = 0;
        while (head + nA < qn && nR + nA < cap) {
            int i = q_req[head + nA];
            int64_t tot = kv_reserve > 0 ? kv_reserve : (int64_t)p[i] + (int64_t)o[i];
            if (reserved + sumTot + tot > kv_budget) break;
            if (!stage_holds(c, sumP, p[i])) break;
            sumTot += tot; sumP += p[i]; ++nA;
        }
        /* 2. decide */
        int prefill;
        int64_t Cp = prefill_us(c, sumP);
        if (nA == 0) prefill = 0;
        else if (nR == 0) prefill = 1;
        else prefill = ((uint64_t)lambda_q16 * (uint64_t)Cd) > (((uint64_t)Cp) << 16);
        if (nA == 0 && nR == 0) { status |= 1; break; }     /* head can never fit: invalid input */

        if (iters == (uint64_t)max_iters) { status |= 1; break; }

        ora_rec rec;
        int64_t dur;
        if (prefill) {
            /* 3. prefill iteration: running decodes stall (PD competition) */
            dur = Cp;
            busy += dur * nA;
            rec.dur_us = (uint32_t)dur; rec.kind_n = 0x80000000u | (uint32_t)nA;
            rec.tokens = (uint32_t)sumP; rec.aux = (uint32_t)head;
            for (int a = 0; a < nA; ++a) {
                int i = q_req[head + a];
                R[nR].kv = p[i]; R[nR].rem = o[i];
                R[nR].total = kv_reserve > 0 ? kv_reserve : (int64_t)p[i] + (int64_t)o[i];
                ++nR;
            }
            head += nA;
            reserved += sumTot;
            Cd = 0;
            ++n_pre;
        } else {
            /* 4. decode iteration: one token for every running request */
            int64_t B = nR, S = 0;
            for (int s = 0; s < nR; ++s) S += R[s].kv;       /* KV lengths before the step */
            dur = ad + bd * B + S / q;
            busy += dur * B;
            int f = 0, w = 0;
            for (int s = 0; s < nR; ++s) {
                R[s].kv += 1; R[s].rem -= 1;
                if (R[s].rem == 0) { reserved -= R[s].total; ++f; }
                else R[w++] = R[s];
            }
            nR = w;
            Cd += dur;
            if (Cd > 2147483647ll) Cd = 2147483647ll;
            rec.dur_us = (uint32_t)dur; rec.kind_n = (uint32_t)B;
            rec.tokens = (uint32_t)S; rec.aux = (uint32_t)f;
            ++n_dec;
        }
        /* 5. clock, trace, hash */
        t += dur;
        if ((int64_t)iters < trace_cap) { if (trace) trace[iters] = rec; }
        else if (trace) status |= 2;
        hash = (hash + (uint64_t)rec.dur_us + ORA_HASH_C1 * rec.kind_n + ORA_HASH_C2 * rec.tokens
                     + ORA_HASH_C3 * rec.aux) * ORA_HASH_M;
        ++iters;
        if (t >= ((int64_t)1 << 39)) { status |= 1; break; }
    }
    res->makespan_us = t;
    res->busy_slot_us = busy;
    res->n_prefill_iters = n_pre;
    res->n_decode_iters = n_dec;
    res->trace_hash = hash;
    res->status = status;
    free(R);
}

/* ------------------------------------------------------------------------- */
/* Algorithm 1, second part: idle clients take the longest request of the     */
/* client with the most remaining tokens                                      */
/* ------------------------------------------------------------------------- */

typedef struct {
    ora_running* R; int nR;
    int32_t* cand; int nA; int64_t sumP, sumTot;   /* claimed, not yet prefilled */
    int ustart, qend;                               /* own queue: unclaimed part [ustart, qend) */
    int64_t remain;                                 /* sum of p+o over the unclaimed part */
    int head;                                       /* requests prefilled so far */
    int64_t reserved, t, busy, Cd;
    uint64_t hash, iters;
    uint32_t n_pre, n_dec;
    int32_t status;
    int finished;
} ora_cstate;

/* o_key: the output lengths the scheduler knows (estimates; o itself when they are exact): the
 * queued tokens of Algorithm 1's remain_token count p + o_key.  kv_reserve as above. */
void ora_simulate_steal(int n, int M, const int32_t* q_off, const int32_t* q_req,
                        const uint32_t* p, const uint32_t* o, const uint32_t* o_key, const ora_cost* c,
                        int cap, int64_t kv_budget, int64_t kv_reserve, uint32_t lambda_q16,
                        uint32_t max_iters,
                        ora_client* res, ora_rec** traces, const int64_t* trace_cap,
                        int32_t* served_by)
{
    const int64_t ad = c->decode_fixed_us,  bd = c->decode_per_seq_us, q = c->decode_kv_div;
    ora_cstate* C = (ora_cstate*)calloc((size_t)M, sizeof(ora_cstate));
    (void)n;
    for (int j = 0; j < M; ++j) {
        C[j].R = (ora_running*)malloc(sizeof(ora_running) * (size_t)cap);
        C[j].cand = (int32_t*)malloc(sizeof(int32_t) * (size_t)cap);
        C[j].ustart = q_off[j]; C[j].qend = q_off[j + 1];
        for (int x = q_off[j]; x < q_off[j + 1]; ++x)
            C[j].remain += (int64_t)p[q_req[x]] + (int64_t)o_key[q_req[x]];
        C[j].hash = ORA_HASH_INIT;
    }
    for (;;) {
        /* the unfinished client with the earliest clock, ties to the lower client */
        int cur = -1;
        for (int j = 0; j < M; ++j)
            if (!C[j].finished && (cur < 0 || C[j].t < C[cur].t)) cur = j;
        if (cur < 0) break;
        ora_cstate* s = &C[cur];

        /* 1. claim from the own queue: a prefix, no skipping */
        while (s->ustart < s->qend && s->nR + s->nA < cap) {
            int i = q_req[s->ustart];
            int64_t tot = kv_reserve > 0 ? kv_reserve : (int64_t)p[i] + (int64_t)o[i];
            if (s->reserved + s->sumTot + tot > kv_budget) break;
            if (!stage_holds(c, s->sumP, p[i])) break;
            s->cand[s->nA++] = i; s->sumTot += tot; s->sumP += p[i];
            s->ustart += 1; s->remain -= (int64_t)p[i] + (int64_t)o_key[i];
            if (served_by) served_by[i] = cur;
        }
        /* 1b. own queue exhausted and a slot free: take the longest waiting request of the client
         *     with the most remaining tokens */
        if (s->ustart == s->qend) {
            while (s->nR + s->nA < cap) {
                int d = -1;
                for (int j = 0; j < M; ++j)
                    if (C[j].remain > 0 && (d < 0 || C[j].remain > C[d].remain)) d = j;
                if (d < 0) break;
                int i = q_req[C[d].ustart];
                int64_t tot = kv_reserve > 0 ? kv_reserve : (int64_t)p[i] + (int64_t)o[i];
                if (s->reserved + s->sumTot + tot > kv_budget) break;
                if (!stage_holds(c, s->sumP, p[i])) break;
                s->cand[s->nA++] = i; s->sumTot += tot; s->sumP += p[i];
                C[d].ustart += 1; C[d].remain -= (int64_t)p[i] + (int64_t)o_key[i];
                if (served_by) served_by[i] = cur;
            }
        }
        if (s->nR == 0 && s->nA == 0) { s->finished = 1; continue; }   /* nothing left anywhere */
        if (s->iters == (uint64_t)max_iters) { s->status |= 1; s->finished = 1; continue; }

        /* 2. decide */
        int64_t Cp = prefill_us(c, s->sumP);
        int prefill;
        if (s->nA == 0) prefill = 0;
        else if (s->nR == 0) prefill = 1;
        else prefill = ((uint64_t)lambda_q16 * (uint64_t)s->Cd) > (((uint64_t)Cp) << 16);

        ora_rec rec;
        int64_t dur;
        if (prefill) {
            dur = Cp;
            s->busy += dur * s->nA;
            rec.dur_us = (uint32_t)dur; rec.kind_n = 0x80000000u | (uint32_t)s->nA;
            rec.tokens = (uint32_t)s->sumP; rec.aux = (uint32_t)s->head;
            for (int a = 0; a < s->nA; ++a) {
                int i = s->cand[a];
                s->R[s->nR].kv = p[i]; s->R[s->nR].rem = o[i];
                s->R[s->nR].total = kv_reserve > 0 ? kv_reserve : (int64_t)p[i] + (int64_t)o[i];
                s->nR += 1;
            }
            s->head += s->nA;
            s->reserved += s->sumTot;
            s->nA = 0; s->sumP = 0; s->sumTot = 0;
            s->Cd = 0;
            s->n_pre += 1;
        } else {
            int64_t B = s->nR, S = 0;
            for (int x = 0; x < s->nR; ++x) S += s->R[x].kv;
            dur = ad + bd * B + S / q;
            s->busy += dur * B;
            int f = 0, w = 0;
            for (int x = 0; x < s->nR; ++x) {
                s->R[x].kv += 1; s->R[x].rem -= 1;
                if (s->R[x].rem == 0) { s->reserved -= s->R[x].total; ++f; }
                else s->R[w++] = s->R[x];
            }
            s->nR = w;
            s->Cd += dur;
            if (s->Cd > 2147483647ll) s->Cd = 2147483647ll;
            rec.dur_us = (uint32_t)dur; rec.kind_n = (uint32_t)B;
            rec.tokens = (uint32_t)S; rec.aux = (uint32_t)f;
            s->n_dec += 1;
        }
        s->t += dur;
        if (traces && traces[cur]) {
            if ((int64_t)s->iters < trace_cap[cur]) traces[cur][s->iters] = rec;
            else s->status |= 2;
        }
        s->hash = (s->hash + (uint64_t)rec.dur_us + ORA_HASH_C1 * rec.kind_n + ORA_HASH_C2 * rec.tokens
                           + ORA_HASH_C3 * rec.aux) * ORA_HASH_M;
        s->iters += 1;
        if (s->t >= ((int64_t)1 << 39)) { s->status |= 1; s->finished = 1; }
    }
    for (int j = 0; j < M; ++j) {
        res[j].makespan_us = C[j].t; res[j].busy_slot_us = C[j].busy;
        res[j].n_prefill_iters = C[j].n_pre; res[j].n_decode_iters = C[j].n_dec;
        res[j].trace_hash = C[j].hash; res[j].status = C[j].status;
        free(C[j].R); free(C[j].cand);
    }
    free(C);
}
