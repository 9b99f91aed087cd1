/*
 * kvpo.c -- CPU oracle for KV-cache placement scoring and annealing.
 *
 * TEST INFRASTRUCTURE, NOT THE PRODUCT. This file is a plain, slow,
 * single-threaded restatement of what the CUDA library computes, written from
 * the paper (arXiv 2508.13231, Section III) and from the integer conventions
 * stated below. It shares no code with the CUDA path and is only ever called
 * by the tests, the smoke check and the benchmark's CPU-baseline leg.
 *
 * Everything is bit-at-a-time and step-at-a-time on purpose: the cost of a
 * schedule is the definition of Eq. 1-4 written out, the annealer takes the
 * moves one after the other in move-index order.
 *
 * Pins (see tests/test_oracle_*.py): Eq. 3-4 worked by hand with the Table I
 * bandwidths, the Unlimited-HBM closed form, the aggregate-bandwidth lower
 * bound, the free-migration per-step optimum, brute force over every static
 * placement and over every dynamic schedule of tiny instances, the published
 * Philox4x32-10 known-answer vectors, incremental-vs-full cost agreement;
 * the proposal decoder against the distribution its definition fixes (swap
 * share, run-length classes, uniform and independent s0, u, v, w) and against
 * proposals decoded by hand from the published Philox blocks.
 * Growing cache (kvpo_set_births; tests/test_oracle_growing.py): a hand-worked
 * instance with H^w / E^w decided by the schedule, the all-HBM and all-DRAM
 * closed forms, the exact reduction to the fixed-population model with the
 * written entries handed over as per-step constants, exhaustive search on
 * tiny instances; the layered trace against the single-layer generator.
 * Parity unpinned: the synthetic trace generator beyond its structural
 * properties (exactly k bits per group and step, lag-1 autocorrelation), and
 * the quality of the annealed bound on large instances (it is only bracketed
 * by the closed-form bounds).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define KVPO_OK 0
#define KVPO_ERR_ARG (-1)
#define KVPO_ERR_CAPACITY (-2)
#define KVPO_ERR_RANGE (-3)
#define KVPO_ERR_NOMEM (-5)

#define MIG_HBM 1u
#define MIG_EXT 2u

#define TAG_MOVE 1u
#define TAG_CALIB 2u
#define TAG_NOISE 3u
#define TAG_BURST 4u

#define TABLE_Q 1024u
#define CALIB_N 1024u

/* ------------------------------------------------------------------ */
/* Philox4x32-10, Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
 * easy as 1, 2, 3" (SC'11), Section 3.3 and the constants of its Table 2:
 * multipliers 0xD2511F53 / 0xCD9E8D57, Weyl key increments 0x9E3779B9 /
 * 0xBB67AE85 (golden ratio and sqrt(3)-1). */
void kvpo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

static void philox(uint64_t seed, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t out[4])
{
    uint32_t ctr[4] = { a, b, c, d };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    kvpo_philox4x32_10(ctr, key, out);
}

/* ------------------------------------------------------------------ */
/* Integer time base: the three bandwidths of Eq. 3-4 reduced to the smallest
 * integer weights with kappa_x proportional to 1/B_x. */
static uint64_t gcd64(uint64_t a, uint64_t b)
{
    while (b) { uint64_t r = a % b; a = b; b = r; }
    return a;
}

/* out = {kappa_h, kappa_k, kappa_d, kappa_e, lcm, gcd} */
int kvpo_tick_weights(uint64_t bw_hbm, uint64_t bw_link, uint64_t bw_dram, uint64_t out[6])
{
    if (!bw_hbm || !bw_link || !bw_dram) return KVPO_ERR_ARG;
    uint64_t g = gcd64(gcd64(bw_hbm, bw_link), bw_dram);
    uint64_t h = bw_hbm / g, k = bw_link / g, d = bw_dram / g;
    uint64_t l = h / gcd64(h, k);
    if (l > (1ull << 40) / k) return KVPO_ERR_RANGE;
    l *= k;
    uint64_t l2 = l / gcd64(l, d);
    if (l2 > (1ull << 40) / d) return KVPO_ERR_RANGE;
    l = l2 * d;
    out[0] = l / h; out[1] = l / k; out[2] = l / d;
    out[3] = out[1] > out[2] ? out[1] : out[2];
    out[4] = l; out[5] = g;
    return KVPO_OK;
}

/* ------------------------------------------------------------------ */
typedef struct kvpo_problem {
    uint32_t U, S, W32, cap;
    uint64_t bytes_per_unit;
    uint64_t kh, kk, kd, ke, lcm, g;
    uint64_t fh, fe;       /* 0/1: migration charged on HBM / on link+DRAM */
    uint32_t *A;           /* [S][W32] */
    uint32_t *a;           /* [S] accessed units per step */
    uint32_t *hw, *ew;     /* [S] */
    uint32_t *birth;       /* [U] or NULL: growing cache, see kvpo_set_births */
    uint32_t *nb;          /* [S] units written (born) during step s */
    double spt;            /* seconds per tick */
} kvpo_problem;

static int bit_of(const uint32_t *row, uint32_t u) { return (int)((row[u >> 5] >> (u & 31)) & 1u); }
static void set_bit(uint32_t *row, uint32_t u, int b)
{
    if (b) row[u >> 5] |= (1u << (u & 31)); else row[u >> 5] &= ~(1u << (u & 31));
}

void kvpo_destroy(kvpo_problem *p)
{
    if (!p) return;
    free(p->A); free(p->a); free(p->hw); free(p->ew); free(p->birth); free(p->nb); free(p);
}

int kvpo_create(kvpo_problem **out, uint32_t units, uint64_t bytes_per_unit, uint32_t steps,
                const uint32_t *access, uint32_t cap, uint64_t bw_hbm, uint64_t bw_link,
                uint64_t bw_dram, uint32_t mig_flags, const uint32_t *hw, const uint32_t *ew)
{
    if (!out || !access || !units || !steps || !bytes_per_unit || cap > units) return KVPO_ERR_ARG;
    uint64_t w[6];
    int rc = kvpo_tick_weights(bw_hbm, bw_link, bw_dram, w);
    if (rc) return rc;
    kvpo_problem *p = (kvpo_problem *)calloc(1, sizeof *p);
    if (!p) return KVPO_ERR_NOMEM;
    p->U = units; p->S = steps; p->W32 = (units + 31) / 32; p->cap = cap;
    p->bytes_per_unit = bytes_per_unit;
    p->kh = w[0]; p->kk = w[1]; p->kd = w[2]; p->ke = w[3]; p->lcm = w[4]; p->g = w[5];
    p->fh = (mig_flags & MIG_HBM) ? 1 : 0;
    p->fe = (mig_flags & MIG_EXT) ? 1 : 0;
    p->spt = (double)bytes_per_unit / ((double)p->lcm * (double)p->g);
    size_t nw = (size_t)steps * p->W32;
    p->A = (uint32_t *)calloc(nw, 4);
    p->a = (uint32_t *)calloc(steps, 4);
    p->hw = (uint32_t *)calloc(steps, 4);
    p->ew = (uint32_t *)calloc(steps, 4);
    if (!p->A || !p->a || !p->hw || !p->ew) { kvpo_destroy(p); return KVPO_ERR_NOMEM; }
    uint64_t mx = 0;
    for (uint32_t s = 0; s < steps; ++s) {
        for (uint32_t u = 0; u < units; ++u) {            /* pad bits are dropped here */
            int b = bit_of(access + (size_t)s * p->W32, u);
            set_bit(p->A + (size_t)s * p->W32, u, b);
            p->a[s] += (uint32_t)b;
        }
        if (hw) p->hw[s] = hw[s];
        if (ew) p->ew[s] = ew[s];
        uint64_t e = (uint64_t)p->hw[s] + p->ew[s];
        if (e > mx) mx = e;
    }
    uint64_t kmax = p->kh > p->ke ? p->kh : p->ke;
    if (kmax * (2ull * units + mx) >= (1ull << 31)) { kvpo_destroy(p); return KVPO_ERR_RANGE; }
    *out = p;
    return KVPO_OK;
}

/* out = {kappa_h, kappa_k, kappa_d, kappa_e, lcm, gcd}; returns seconds per tick */
double kvpo_get_weights(const kvpo_problem *p, uint64_t out[6])
{
    out[0] = p->kh; out[1] = p->kk; out[2] = p->kd; out[3] = p->ke; out[4] = p->lcm; out[5] = p->g;
    return p->spt;
}

/*
 * Growing cache (Section III-A lists the newly written entries H^w and E^w among
 * the scheduling decisions). birth[u] = 0: unit u exists before the first step
 * (written by the prefill, outside the model). birth[u] = b >= 1: unit u is
 * written during step b; before b it is nowhere, so its placement bits of
 * earlier steps are ignored and it may not be accessed there. At step b the
 * placement bit decides where the new entry goes: set = written to HBM (it
 * counts in |H^w_b|), clear = written to off-package DRAM (|E^w_b|). Being
 * written is not a migration. The caller's hw/ew constants still add.
 */
int kvpo_set_births(kvpo_problem *p, const uint32_t *birth)
{
    if (!p || !birth || p->birth) return KVPO_ERR_ARG;
    uint32_t *b = (uint32_t *)malloc((size_t)p->U * 4);
    uint32_t *nb = (uint32_t *)calloc(p->S, 4);
    if (!b || !nb) { free(b); free(nb); return KVPO_ERR_NOMEM; }
    for (uint32_t u = 0; u < p->U; ++u) {
        if (birth[u] >= p->S) { free(b); free(nb); return KVPO_ERR_ARG; }
        b[u] = birth[u];
        if (birth[u]) ++nb[birth[u]];
        for (uint32_t s = 0; s < birth[u]; ++s)
            if (bit_of(p->A + (size_t)s * p->W32, u)) { free(b); free(nb); return KVPO_ERR_ARG; }
    }
    uint64_t mx = 0;
    for (uint32_t s = 0; s < p->S; ++s) {
        uint64_t e = (uint64_t)p->hw[s] + p->ew[s] + nb[s];
        if (e > mx) mx = e;
    }
    uint64_t kmax = p->kh > p->ke ? p->kh : p->ke;
    if (kmax * (2ull * p->U + mx) >= (1ull << 31)) { free(b); free(nb); return KVPO_ERR_RANGE; }
    p->birth = b; p->nb = nb;
    return KVPO_OK;
}

static int alive(const kvpo_problem *p, uint32_t u, uint32_t s) { return !p->birth || p->birth[u] <= s; }
static int born_at(const kvpo_problem *p, uint32_t u, uint32_t s) { return p->birth && s > 0 && p->birth[u] == s; }

/* Eq. 2-4 for one step, in ticks. hr: accessed units resident in HBM,
 * mi / mo: units migrated into / out of HBM before this step, hb: units
 * written to HBM at birth during this step (0 without kvpo_set_births). */
static uint64_t step_cost(const kvpo_problem *p, uint32_t s, uint64_t hr, uint64_t mi, uint64_t mo, uint64_t hb)
{
    uint64_t hw = p->hw[s] + hb;                                             /* |H^w| */
    uint64_t ew = p->ew[s] + (p->nb ? p->nb[s] - hb : 0);                    /* |E^w| */
    uint64_t er = (uint64_t)p->a[s] - hr;                                    /* |E^r| */
    uint64_t th = p->kh * (hr + hw + p->fh * (mi + mo));                     /* Eq. 3 */
    uint64_t w1 = p->kk * (ew + p->fe * mo);                                 /* link, outbound  */
    uint64_t w2 = p->kk * (p->fe * mi);                                      /* link, inbound   */
    uint64_t w3 = p->kd * (ew + p->fe * (mi + mo));                          /* DRAM channels   */
    uint64_t wm = w1 > w2 ? w1 : w2;
    if (w3 > wm) wm = w3;
    uint64_t te = p->ke * er + wm;                                           /* Eq. 4 */
    return th > te ? th : te;                                                /* Eq. 2 */
}

/* The cardinalities of step s of schedule P (rows of W32 words): hr, mi, mo, occ and, for a growing cache, hb.
 * A unit that does not exist yet counts as absent whatever its bit says. */
static void step_counts(const kvpo_problem *p, const uint32_t *P, uint32_t s, uint32_t c[5])
{
    const uint32_t *row = P + (size_t)s * p->W32;
    const uint32_t *prev = s ? row - p->W32 : row;                           /* P[-1] := P[0] */
    const uint32_t *acc = p->A + (size_t)s * p->W32;
    c[0] = c[1] = c[2] = c[3] = c[4] = 0;
    for (uint32_t u = 0; u < p->U; ++u) {
        int pb = bit_of(row, u) & alive(p, u, s);
        int qb = s ? (bit_of(prev, u) & alive(p, u, s - 1)) : pb;
        int ab = bit_of(acc, u);
        c[0] += (uint32_t)(pb & ab);               /* hr  */
        c[3] += (uint32_t)pb;                      /* occ */
        if (born_at(p, u, s)) {
            c[4] += (uint32_t)pb;                  /* hb: written to HBM, not migrated */
        } else {
            c[1] += (uint32_t)(pb & (1 - qb));     /* mi  */
            c[2] += (uint32_t)((1 - pb) & qb);     /* mo  */
        }
    }
}

/*
 * Eq. 1-5 for one schedule. Any output pointer may be NULL.
 * counts: [S][4] = {hr, mi, mo, occ}. Returns the first infeasible step or -1
 * through *bad_step.
 */
int kvpo_eval(const kvpo_problem *p, const uint32_t *P, uint64_t *step_ticks, uint64_t *total_ticks,
              double *step_seconds, double *total_seconds, int32_t *bad_step, uint32_t *counts)
{
    if (!p || !P) return KVPO_ERR_ARG;
    uint64_t T = 0;
    int32_t bad = -1;
    for (uint32_t s = 0; s < p->S; ++s) {
        uint32_t c[5];
        step_counts(p, P, s, c);
        uint64_t f = step_cost(p, s, c[0], c[1], c[2], c[4]);
        if (c[3] > p->cap && bad < 0) bad = (int32_t)s;                      /* Eq. 5 */
        if (step_ticks) step_ticks[s] = f;
        if (step_seconds) step_seconds[s] = (double)f * p->spt;
        if (counts) memcpy(counts + 4 * (size_t)s, c, 4 * sizeof c[0]);
        T += f;                                                              /* Eq. 1 */
    }
    if (total_ticks) *total_ticks = T;
    if (total_seconds) *total_seconds = (double)T * p->spt;
    if (bad_step) *bad_step = bad;
    return KVPO_OK;
}

/* hb [S]: units written to HBM at birth in every step (all 0 for a fixed population). */
int kvpo_eval_hb(const kvpo_problem *p, const uint32_t *P, uint32_t *hb)
{
    if (!p || !P || !hb) return KVPO_ERR_ARG;
    for (uint32_t s = 0; s < p->S; ++s) {
        uint32_t c[5];
        step_counts(p, P, s, c);
        hb[s] = c[4];
    }
    return KVPO_OK;
}

/* ------------------------------------------------------------------ */
/* Initial placements. mode 0: units 0..cap-1 (Static Placement: fill HBM in
 * arrival order, never migrate). mode 1: the cap most accessed units, ties to
 * the lower index. The same row is used at every step; in a growing cache a
 * unit of the row enters HBM when it is written. */
int kvpo_init_placement(const kvpo_problem *p, uint32_t mode, uint32_t *P)
{
    if (!p || !P || mode > 1) return KVPO_ERR_ARG;
    uint32_t *row = (uint32_t *)calloc(p->W32, 4);
    if (!row) return KVPO_ERR_NOMEM;
    if (mode == 0) {
        for (uint32_t u = 0; u < p->cap; ++u) set_bit(row, u, 1);
    } else {
        uint32_t *cnt = (uint32_t *)calloc(p->U, 4);
        if (!cnt) { free(row); return KVPO_ERR_NOMEM; }
        uint32_t cmax = 0;
        for (uint32_t u = 0; u < p->U; ++u) {
            for (uint32_t s = 0; s < p->S; ++s) cnt[u] += (uint32_t)bit_of(p->A + (size_t)s * p->W32, u);
            if (cnt[u] > cmax) cmax = cnt[u];
        }
        /* walk the counts from high to low, units in index order within a count */
        uint32_t placed = 0;
        for (int64_t c = cmax; c >= 0 && placed < p->cap; --c)
            for (uint32_t u = 0; u < p->U && placed < p->cap; ++u)
                if (cnt[u] == (uint32_t)c) { set_bit(row, u, 1); ++placed; }
        free(cnt);
    }
    for (uint32_t s = 0; s < p->S; ++s) {
        memset(P + (size_t)s * p->W32, 0, (size_t)p->W32 * 4);
        for (uint32_t u = 0; u < p->U; ++u)
            set_bit(P + (size_t)s * p->W32, u, bit_of(row, u) & alive(p, u, s));
    }
    free(row);
    return KVPO_OK;
}

/* ------------------------------------------------------------------ */
/* Quantised Metropolis thresholds (Section III-B: P(accept) = exp(-dT/C)). */
int kvpo_accept_table(const double *temps, uint32_t levels, uint32_t *table, uint32_t *shifts)
{
    if (!temps || !table || !shifts || !levels) return KVPO_ERR_ARG;
    for (uint32_t j = 0; j < levels; ++j) {
        double C = temps[j];
        if (!(C >= 1.0)) C = 1.0;
        uint32_t sh = 0;
        while ((double)TABLE_Q * (double)(1ull << sh) < 23.0 * C) {
            ++sh;
            if (sh > 40) return KVPO_ERR_RANGE;
        }
        shifts[j] = sh;
        for (uint32_t q = 0; q < TABLE_Q; ++q) {
            double mid = ((double)q + 0.5) * (double)(1ull << sh);
            double v = 4294967296.0 * exp(-mid / C);
            table[(size_t)j * TABLE_Q + q] = v >= 4294967295.0 ? 0xFFFFFFFFu : (uint32_t)v;
        }
    }
    return KVPO_OK;
}

/* ------------------------------------------------------------------ */
typedef struct {
    uint32_t chains, levels;
    uint64_t moves, seed;
    double p0, alpha;
    const double *temps;
    uint32_t early_stop_permille, early_stop_from_level;
    uint32_t init_mode, p_swap_256, max_len_log2, first_chain;
    const uint32_t *init_schedule;
} kvpo_anneal_params;

typedef struct {
    uint64_t best_ticks, best_move, final_ticks, moves_done;
    uint64_t n_accepted, n_changed, n_infeasible, traj_hash;
} kvpo_chain_result;

typedef struct {
    int swap;            /* 1: exchange placement of u and v; 0: flip placement of u */
    uint32_t s0, len;    /* steps s0 .. s0+len-1 (clipped to the horizon) */
    uint32_t u, v;
    uint32_t w;          /* uniform for the Metropolis test */
} move_t;

/* Proposal for (chain, move index): one Philox block decides everything. */
static move_t decode_move(const kvpo_problem *p, const kvpo_anneal_params *ap,
                          uint64_t m, uint32_t chain, uint32_t tag)
{
    uint32_t r[4];
    philox(ap->seed, (uint32_t)m, (uint32_t)(m >> 32), chain, tag, r);
    move_t mv;
    mv.swap = (r[0] & 255u) < ap->p_swap_256;
    uint32_t k = (((r[0] >> 8) & 255u) * (ap->max_len_log2 + 1u)) >> 8;
    mv.len = (1u << k) < 30u ? (1u << k) : 30u;
    mv.s0 = ((r[0] >> 16) * p->S) >> 16;
    mv.u = (uint32_t)(((uint64_t)r[1] * p->U) >> 32);
    mv.v = (uint32_t)(((uint64_t)r[2] * p->U) >> 32);
    mv.w = r[3];
    return mv;
}

/*
 * Test access to the proposal decoder: the proposals of moves m_begin ..
 * m_begin+count-1 of `chain` under counter tag `tag`, as the annealer draws them.
 *   out [count][6] = {swap, s0, len, u, v, w}
 */
int kvpo_decode_moves(const kvpo_problem *p, const kvpo_anneal_params *ap, uint32_t chain, uint32_t tag,
                      uint64_t m_begin, uint32_t count, uint32_t *out)
{
    if (!p || !ap || !out) return KVPO_ERR_ARG;
    for (uint32_t i = 0; i < count; ++i) {
        move_t mv = decode_move(p, ap, m_begin + i, chain, tag);
        uint32_t *o = out + (size_t)i * 6;
        o[0] = (uint32_t)mv.swap; o[1] = mv.s0; o[2] = mv.len; o[3] = mv.u; o[4] = mv.v; o[5] = mv.w;
    }
    return KVPO_OK;
}

typedef struct {
    uint32_t *P;                    /* [S][W32] current schedule (bits of unborn units stay clear) */
    uint32_t *hr, *mi, *mo, *occ;   /* [S] */
    uint32_t *hb;                   /* [S] units written to HBM at birth */
    uint64_t cur;
} chain_state;

/* Placement bit unit x would have at step t if the move were applied. A move
 * acts on a step only if the units it names exist there. */
static int proposed_bit(const kvpo_problem *p, const chain_state *st, const move_t *mv, uint32_t t, uint32_t x)
{
    const uint32_t *row = st->P + (size_t)t * p->W32;
    int in_range = t >= mv->s0 && t < mv->s0 + mv->len && alive(p, mv->u, t) && (!mv->swap || alive(p, mv->v, t));
    if (!in_range) return bit_of(row, x);
    if (!mv->swap) return x == mv->u ? !bit_of(row, x) : bit_of(row, x);
    if (x == mv->u) return bit_of(row, mv->v);
    if (x == mv->v) return bit_of(row, mv->u);
    return bit_of(row, x);
}

/*
 * Evaluate a proposal against the current state without applying it.
 * Returns 0 = evaluated, 1 = infeasible (a flip would exceed capacity).
 * d[t - s0][0..4] receive the changes of hr, mi, mo, occ, hb of every affected
 * step t = s0 .. last, where last = min(s0 + len, S - 1): the step after the
 * run is affected too because its migration counts compare against the run's
 * last row.
 */
static int evaluate_move(const kvpo_problem *p, const chain_state *st, const move_t *mv,
                         int64_t *delta, int32_t d[32][5], uint32_t *last_out, int *changed)
{
    uint32_t last = mv->s0 + mv->len;
    if (last > p->S - 1) last = p->S - 1;
    *last_out = last;
    *changed = 0;
    uint32_t xs[2] = { mv->u, mv->v };
    int nx = (mv->swap && mv->v != mv->u) ? 2 : 1;
    int64_t dsum = 0;
    for (uint32_t t = mv->s0; t <= last; ++t) {
        int32_t *dt = d[t - mv->s0];
        dt[0] = dt[1] = dt[2] = dt[3] = dt[4] = 0;
        for (int i = 0; i < nx; ++i) {
            uint32_t x = xs[i];
            int po = bit_of(st->P + (size_t)t * p->W32, x);
            int pn = proposed_bit(p, st, mv, t, x);
            int qo = t ? bit_of(st->P + (size_t)(t - 1) * p->W32, x) : po;
            int qn = t ? proposed_bit(p, st, mv, t - 1, x) : pn;
            int ab = bit_of(p->A + (size_t)t * p->W32, x);
            dt[0] += ab * (pn - po);
            dt[3] += pn - po;
            if (born_at(p, x, t)) {
                dt[4] += pn - po;                     /* written to HBM instead of DRAM, or back */
            } else {
                dt[1] += (pn & (1 - qn)) - (po & (1 - qo));
                dt[2] += ((1 - pn) & qn) - ((1 - po) & qo);
            }
            if (pn != po) *changed = 1;
        }
        if (!mv->swap && (int64_t)st->occ[t] + dt[3] > (int64_t)p->cap && dt[3] > 0) return 1;
        uint64_t f_old = step_cost(p, t, st->hr[t], st->mi[t], st->mo[t], st->hb[t]);
        uint64_t f_new = step_cost(p, t, (uint64_t)((int64_t)st->hr[t] + dt[0]),
                                   (uint64_t)((int64_t)st->mi[t] + dt[1]),
                                   (uint64_t)((int64_t)st->mo[t] + dt[2]),
                                   (uint64_t)((int64_t)st->hb[t] + dt[4]));
        dsum += (int64_t)f_new - (int64_t)f_old;
    }
    *delta = dsum;
    return 0;
}

static void apply_move(const kvpo_problem *p, chain_state *st, const move_t *mv,
                       int32_t d[32][5], uint32_t last, int64_t delta)
{
    for (uint32_t t = mv->s0; t < mv->s0 + mv->len && t < p->S; ++t) {
        uint32_t *row = st->P + (size_t)t * p->W32;
        int bu = proposed_bit(p, st, mv, t, mv->u);
        int bv = mv->swap ? proposed_bit(p, st, mv, t, mv->v) : 0;
        set_bit(row, mv->u, bu);
        if (mv->swap) set_bit(row, mv->v, bv);
    }
    for (uint32_t t = mv->s0; t <= last; ++t) {
        int32_t *dt = d[t - mv->s0];
        st->hr[t] = (uint32_t)((int32_t)st->hr[t] + dt[0]);
        st->mi[t] = (uint32_t)((int32_t)st->mi[t] + dt[1]);
        st->mo[t] = (uint32_t)((int32_t)st->mo[t] + dt[2]);
        st->occ[t] = (uint32_t)((int32_t)st->occ[t] + dt[3]);
        st->hb[t] = (uint32_t)((int32_t)st->hb[t] + dt[4]);
    }
    st->cur = (uint64_t)((int64_t)st->cur + delta);
}

static int state_init(const kvpo_problem *p, chain_state *st, const uint32_t *P0)
{
    size_t nw = (size_t)p->S * p->W32;
    st->P = (uint32_t *)malloc(nw * 4);
    st->hr = (uint32_t *)malloc((size_t)p->S * 4);
    st->mi = (uint32_t *)malloc((size_t)p->S * 4);
    st->mo = (uint32_t *)malloc((size_t)p->S * 4);
    st->occ = (uint32_t *)malloc((size_t)p->S * 4);
    st->hb = (uint32_t *)malloc((size_t)p->S * 4);
    if (!st->P || !st->hr || !st->mi || !st->mo || !st->occ || !st->hb) return KVPO_ERR_NOMEM;
    memcpy(st->P, P0, nw * 4);
    st->cur = 0;
    for (uint32_t s = 0; s < p->S; ++s) {
        uint32_t c[5];
        step_counts(p, st->P, s, c);
        st->hr[s] = c[0]; st->mi[s] = c[1]; st->mo[s] = c[2]; st->occ[s] = c[3]; st->hb[s] = c[4];
        if (c[3] > p->cap) return KVPO_ERR_CAPACITY;
        st->cur += step_cost(p, s, c[0], c[1], c[2], c[4]);
    }
    return KVPO_OK;
}

static void state_free(chain_state *st)
{
    free(st->P); free(st->hr); free(st->mi); free(st->mo); free(st->occ); free(st->hb);
}

/* Resolve the initial schedule named by the parameters into P0 [S][W32]. */
static int resolve_init(const kvpo_problem *p, const kvpo_anneal_params *ap, uint32_t *P0)
{
    if (ap->init_mode == 2) {
        if (!ap->init_schedule) return KVPO_ERR_ARG;
        memset(P0, 0, (size_t)p->S * p->W32 * 4);
        for (uint32_t s = 0; s < p->S; ++s)
            for (uint32_t u = 0; u < p->U; ++u)
                set_bit(P0 + (size_t)s * p->W32, u, bit_of(ap->init_schedule + (size_t)s * p->W32, u) & alive(p, u, s));
        return KVPO_OK;
    }
    return kvpo_init_placement(p, ap->init_mode, P0);
}

/*
 * Temperature ladder when the caller gives none: 1024 calibration proposals
 * are evaluated (never applied) at the initial state; C_0 is chosen so that an
 * uphill move of their mean size is accepted with probability p0, and
 * C_{j+1} = alpha * C_j (Section III-B: p0 = 0.8, alpha = 0.9).
 * temps_out [levels]; *mean_out = the integer mean of the positive deltas.
 */
int kvpo_default_temps(const kvpo_problem *p, const kvpo_anneal_params *ap, double *temps_out, uint64_t *mean_out)
{
    if (!p || !ap || !temps_out) return KVPO_ERR_ARG;
    if (!(ap->p0 > 0.0 && ap->p0 < 1.0) || !(ap->alpha > 0.0 && ap->alpha <= 1.0)) return KVPO_ERR_ARG;
    uint32_t *P0 = (uint32_t *)malloc((size_t)p->S * p->W32 * 4);
    if (!P0) return KVPO_ERR_NOMEM;
    int rc = resolve_init(p, ap, P0);
    chain_state st;
    memset(&st, 0, sizeof st);
    if (!rc) rc = state_init(p, &st, P0);
    if (rc) { state_free(&st); free(P0); return rc; }
    uint64_t sum = 0, cnt = 0;
    for (uint32_t i = 0; i < CALIB_N; ++i) {
        move_t mv = decode_move(p, ap, i, 0, TAG_CALIB);
        int64_t delta; int32_t d[32][5]; uint32_t last; int changed;
        if (evaluate_move(p, &st, &mv, &delta, d, &last, &changed)) continue;
        if (delta > 0) { sum += (uint64_t)delta; ++cnt; }
    }
    uint64_t mean = cnt ? sum / cnt : 1;
    if (mean == 0) mean = 1;
    if (mean_out) *mean_out = mean;
    double C = -(double)mean / log(ap->p0);
    for (uint32_t j = 0; j < ap->levels; ++j) { temps_out[j] = C; C = C * ap->alpha; }
    state_free(&st); free(P0);
    return KVPO_OK;
}

/*
 * Run chains chain_begin .. chain_begin+chain_count-1, each for at most
 * `upto_moves` proposals (pass ap->moves for a full run; level boundaries are
 * always those of the full budget ap->moves).
 *   results      [chain_count]
 *   final_states [chain_count][S][W32] or NULL : schedule after the last move
 *   best_states  [chain_count][S][W32] or NULL : schedule when best_ticks was reached
 */
int kvpo_anneal_chains(const kvpo_problem *p, const kvpo_anneal_params *ap,
                       const uint32_t *table, const uint32_t *shifts,
                       uint32_t chain_begin, uint32_t chain_count, uint64_t upto_moves,
                       kvpo_chain_result *results, uint32_t *final_states, uint32_t *best_states)
{
    if (!p || !ap || !table || !shifts || !results) return KVPO_ERR_ARG;
    if (!ap->levels || !ap->moves || ap->p_swap_256 > 256 || ap->max_len_log2 > 5) return KVPO_ERR_ARG;
    size_t nw = (size_t)p->S * p->W32;
    uint32_t *P0 = (uint32_t *)malloc(nw * 4);
    if (!P0) return KVPO_ERR_NOMEM;
    int rc = resolve_init(p, ap, P0);
    if (rc) { free(P0); return rc; }
    uint64_t per_level = ap->moves / ap->levels;
    if (per_level == 0) per_level = 1;
    if (upto_moves > ap->moves) upto_moves = ap->moves;

    for (uint32_t ci = 0; ci < chain_count; ++ci) {
        uint32_t chain = chain_begin + ci;
        chain_state st;
        memset(&st, 0, sizeof st);
        rc = state_init(p, &st, P0);
        if (rc) { state_free(&st); free(P0); return rc; }
        kvpo_chain_result r;
        memset(&r, 0, sizeof r);
        r.best_ticks = st.cur;
        r.best_move = UINT64_MAX;
        if (best_states) memcpy(best_states + ci * nw, st.P, nw * 4);
        uint64_t best_at_boundary = st.cur;
        uint64_t m = 0;
        for (; m < upto_moves; ++m) {
            uint64_t lev = m / per_level;
            if (lev > ap->levels - 1) lev = ap->levels - 1;
            /* termination rule of Section III-B, checked when a new level starts */
            if (m > 0 && m % per_level == 0 && m / per_level <= ap->levels - 1) {
                if (ap->early_stop_permille && lev >= ap->early_stop_from_level &&
                    (best_at_boundary - r.best_ticks) * 1000ull < best_at_boundary * (uint64_t)ap->early_stop_permille)
                    break;
                best_at_boundary = r.best_ticks;
            }
            move_t mv = decode_move(p, ap, m, chain, TAG_MOVE);
            int64_t delta; int32_t d[32][5]; uint32_t last; int changed;
            if (evaluate_move(p, &st, &mv, &delta, d, &last, &changed)) { ++r.n_infeasible; continue; }
            int accept;
            if (delta <= 0) accept = 1;                                 /* downhill or level: always */
            else {
                uint64_t q = (uint64_t)delta >> shifts[lev];
                accept = q < TABLE_Q && mv.w < table[lev * TABLE_Q + q];   /* Metropolis */
            }
            if (!accept) continue;
            ++r.n_accepted;
            if (!changed) continue;
            apply_move(p, &st, &mv, d, last, delta);
            ++r.n_changed;
            r.traj_hash = (r.traj_hash ^ m) * 0x9E3779B97F4A7C15ull + st.cur;
            if (st.cur < r.best_ticks) {
                r.best_ticks = st.cur;
                r.best_move = m;
                if (best_states) memcpy(best_states + ci * nw, st.P, nw * 4);
            }
        }
        r.moves_done = m;
        r.final_ticks = st.cur;
        if (final_states) memcpy(final_states + ci * nw, st.P, nw * 4);
        results[ci] = r;
        state_free(&st);
    }
    free(P0);
    return KVPO_OK;
}

/*
 * The whole search: chains first_chain .. first_chain+chains-1 in index order, the bound = the lowest
 * best_ticks, ties to the lower chain index; best_schedule [S][W32] receives the
 * winner's schedule at the moment it reached the bound. per_chain [chains] or NULL.
 */
int kvpo_anneal(const kvpo_problem *p, const kvpo_anneal_params *ap, const uint32_t *table,
                const uint32_t *shifts, uint32_t *best_schedule, uint64_t *best_ticks,
                uint32_t *best_chain, kvpo_chain_result *per_chain)
{
    if (!p || !ap || !ap->chains) return KVPO_ERR_ARG;
    size_t nw = (size_t)p->S * p->W32;
    uint32_t *tmp = (uint32_t *)malloc(nw * 4);
    if (!tmp) return KVPO_ERR_NOMEM;
    uint64_t bt = UINT64_MAX; uint32_t bc = 0;
    for (uint32_t i = 0; i < ap->chains; ++i) {
        uint32_t c = ap->first_chain + i;
        kvpo_chain_result r;
        int rc = kvpo_anneal_chains(p, ap, table, shifts, c, 1, ap->moves, &r, NULL, tmp);
        if (rc) { free(tmp); return rc; }
        if (per_chain) per_chain[i] = r;
        if (r.best_ticks < bt) {
            bt = r.best_ticks; bc = c;
            if (best_schedule) memcpy(best_schedule, tmp, nw * 4);
        }
    }
    if (best_ticks) *best_ticks = bt;
    if (best_chain) *best_chain = bc;
    free(tmp);
    return KVPO_OK;
}

/* Full recomputation of a chain state's counters and cost; used by the
 * invariant tests: returns 0 when the schedule's Eq. 1 total equals `ticks`. */
int kvpo_check_total(const kvpo_problem *p, const uint32_t *P, uint64_t ticks)
{
    uint64_t T; int32_t bad;
    kvpo_eval(p, P, NULL, &T, NULL, NULL, &bad, NULL);
    return (T == ticks && bad < 0) ? 0 : 1;
}

/* ------------------------------------------------------------------ */
/* Synthetic access traces (stand-in for recorded attention scores, Section
 * IV-A; the paper's own synthesised traces of Section IV-B are unspecified). */
typedef struct {
    uint32_t groups, units_per_group, steps, topk;
    uint64_t seed;
    int32_t rho_q, c_q, sigma_q, burst_jump;
    uint32_t burst_thr, reserved;
    const int32_t *base;
    uint32_t layers, reserved2;   /* 0 or 1: every group reads at every step */
    const uint32_t *birth;        /* [U] or NULL: step from which a unit can be read */
} kvpo_trace_params;

static int64_t floor_shift16(int64_t v)
{
    /* floor(v / 65536) for either sign */
    int64_t q = v / 65536;
    if (v % 65536 != 0 && v < 0) --q;
    return q;
}

/*
 * Groups group_begin .. group_begin+group_count-1 only (groups are independent);
 * bits of other groups are left 0. scores_out: [steps][U] int32 or NULL (for
 * statistical tests; only the selected groups are written).
 *
 * layers = L > 1: the steps are the (token n, layer l) pairs of Section III-A in
 * the order s = n * L + l. The groups are split into L consecutive blocks, one
 * per layer; a group reads only at the steps of its layer, and the importance
 * of its units advances once per token (the noise counter is (u, n)). With
 * birth given, a group reads its min(topk, existing) most important existing
 * units (birth[u] <= s).
 */
int kvpo_trace_generate(const kvpo_trace_params *tp, uint32_t group_begin, uint32_t group_count,
                        uint32_t *access, int32_t *scores_out)
{
    if (!tp || !access || !tp->groups || !tp->units_per_group || !tp->steps) return KVPO_ERR_ARG;
    if (!tp->topk || tp->topk > tp->units_per_group) return KVPO_ERR_ARG;
    if (group_begin > tp->groups || group_count > tp->groups - group_begin) return KVPO_ERR_ARG;
    if (tp->layers > 1 && tp->groups % tp->layers) return KVPO_ERR_ARG;
    if (tp->rho_q < 0 || tp->rho_q > 65536 || tp->c_q < 0 || tp->c_q > (1 << 20) ||
        tp->sigma_q < 0 || tp->sigma_q > (1 << 20)) return KVPO_ERR_ARG;
    uint64_t U64 = (uint64_t)tp->groups * tp->units_per_group;
    if (U64 >= (1ull << 26)) return KVPO_ERR_RANGE;
    uint32_t U = (uint32_t)U64, n = tp->units_per_group, W32 = (U + 31) / 32;
    /* scores must stay inside int32: bound |x_t| step by step */
    {
        int64_t emax = floor_shift16((int64_t)262140 * 80265) + 1;
        int64_t jump = tp->burst_thr ? llabs((int64_t)tp->burst_jump) : 0;
        int64_t b = floor_shift16((int64_t)tp->sigma_q * emax) + 1 + jump;
        for (uint32_t t = 1; t < tp->steps; ++t) {
            b = floor_shift16((int64_t)tp->rho_q * b + (int64_t)tp->c_q * emax) + 1 + jump;
            if (b >= (1ll << 30)) return KVPO_ERR_RANGE;
        }
        if (b >= (1ll << 30)) return KVPO_ERR_RANGE;
        if (tp->base)
            for (uint32_t u = 0; u < U; ++u)
                if (tp->base[u] > (1 << 29) || tp->base[u] < -(1 << 29)) return KVPO_ERR_RANGE;
    }
    int64_t *x = (int64_t *)calloc(U, sizeof(int64_t));
    int64_t *score = (int64_t *)calloc(n, sizeof(int64_t));
    uint8_t *picked = (uint8_t *)calloc(n, 1);
    if (!x || !score || !picked) { free(x); free(score); free(picked); return KVPO_ERR_NOMEM; }
    memset(access, 0, (size_t)tp->steps * W32 * 4);
    uint32_t L = tp->layers ? tp->layers : 1;
    uint32_t per_layer = tp->groups / L;
    for (uint32_t t = 0; t < tp->steps; ++t) {
        uint32_t tok = t / L, layer = t % L;
        for (uint32_t g = group_begin; g < group_begin + group_count; ++g) {
            if (g / per_layer != layer) continue;
            for (uint32_t i = 0; i < n; ++i) {
                uint32_t u = g * n + i;
                uint32_t r[4];
                philox(tp->seed, u, tok, 0, TAG_NOISE, r);
                int64_t sum = 0;
                for (int k = 0; k < 4; ++k) sum += (int64_t)(r[k] & 0xFFFFu) + (int64_t)(r[k] >> 16);
                int64_t e = floor_shift16((sum - 262140) * 80265);
                if (tok == 0) x[u] = floor_shift16((int64_t)tp->sigma_q * e);
                else x[u] = floor_shift16((int64_t)tp->rho_q * x[u] + (int64_t)tp->c_q * e);
                if (tp->burst_thr) {
                    philox(tp->seed, u, tok, 0, TAG_BURST, r);
                    if (r[0] < tp->burst_thr) x[u] += tp->burst_jump;
                }
            }
            uint32_t existing = 0;
            for (uint32_t i = 0; i < n; ++i) {
                uint32_t u = g * n + i;
                score[i] = x[u] + (tp->base ? tp->base[u] : 0);
                picked[i] = (uint8_t)(tp->birth && tp->birth[u] > t);    /* not there yet: never chosen */
                existing += !picked[i];
                if (scores_out) scores_out[(size_t)t * U + u] = (int32_t)score[i];
            }
            /* k rounds of "largest remaining score, lowest index among equals" */
            uint32_t k = tp->topk < existing ? tp->topk : existing;
            for (uint32_t r = 0; r < k; ++r) {
                uint32_t arg = n;
                for (uint32_t i = 0; i < n; ++i)
                    if (!picked[i] && (arg == n || score[i] > score[arg])) arg = i;
                picked[arg] = 1;
                set_bit(access + (size_t)t * W32, g * n + arg, 1);
            }
        }
    }
    free(x); free(score); free(picked);
    return KVPO_OK;
}

/* ------------------------------------------------------------------ */
/* Placement policies that produce a schedule from the access pattern (Section IV-A's comparison strategies and
 * the look-ahead policy of Section III-B that the paper's annealer tunes). Each starts from the static placement
 * named by init_mode (0: units 0..cap-1, the paper's Static Placement; 1: the cap most accessed units) and
 * writes P [S][W32]. Migrations decided "at step s" are in place when step s reads (they are charged to step s by
 * the cost model; at s = 0 they are free because P[-1] := P[0]). */

typedef struct { uint32_t f, u; } fu_t;

static int by_freq_desc(const void *a, const void *b)
{
    const fu_t *x = (const fu_t *)a, *y = (const fu_t *)b;
    if (x->f != y->f) return x->f > y->f ? -1 : 1;
    return x->u < y->u ? -1 : (x->u > y->u ? 1 : 0);
}

static int by_freq_asc(const void *a, const void *b)
{
    const fu_t *x = (const fu_t *)a, *y = (const fu_t *)b;
    if (x->f != y->f) return x->f < y->f ? -1 : 1;
    return x->u < y->u ? -1 : (x->u > y->u ? 1 : 0);
}

/*
 * Look-ahead policy with window W (steps) and migration ratio R = ratio_permille / 1000 (Section III-B).
 * Before step s: every unit's frequency is the number of its accesses in steps s .. s+W-1. The units that are
 * not in HBM and will be accessed are the candidates, ranked by frequency (ties: lower index); only the top
 * floor(R * candidates) of them may migrate. They first fill free HBM capacity; after that the j-th remaining
 * candidate replaces the j-th resident in order of rising frequency (ties: lower index), as long as that resident
 * is accessed less often than the candidate.
 */
int kvpo_policy_lookahead(const kvpo_problem *p, uint32_t init_mode, uint32_t W, uint32_t ratio_permille, uint32_t *P)
{
    if (p && p->birth) return KVPO_ERR_ARG;       /* the policies are defined on a fixed population */
    if (!p || !P || init_mode > 1 || W < 1 || W > 64 || ratio_permille > 1000) return KVPO_ERR_ARG;
    int rc = kvpo_init_placement(p, init_mode, P);
    if (rc) return rc;
    uint8_t *in = (uint8_t *)calloc(p->U, 1);
    fu_t *cand = (fu_t *)malloc(sizeof(fu_t) * p->U), *res = (fu_t *)malloc(sizeof(fu_t) * p->U);
    if (!in || !cand || !res) { free(in); free(cand); free(res); return KVPO_ERR_NOMEM; }
    for (uint32_t u = 0; u < p->U; ++u) in[u] = (uint8_t)bit_of(P, u);
    for (uint32_t s = 0; s < p->S; ++s) {
        uint32_t nc = 0, nr = 0;
        for (uint32_t u = 0; u < p->U; ++u) {
            uint32_t f = 0;
            for (uint32_t t = s; t < s + W && t < p->S; ++t) f += (uint32_t)bit_of(p->A + (size_t)t * p->W32, u);
            if (in[u]) { res[nr].f = f; res[nr].u = u; ++nr; }
            else if (f > 0) { cand[nc].f = f; cand[nc].u = u; ++nc; }
        }
        qsort(cand, nc, sizeof(fu_t), by_freq_desc);
        qsort(res, nr, sizeof(fu_t), by_freq_asc);
        uint32_t k = (uint32_t)(((uint64_t)nc * ratio_permille) / 1000u);
        uint32_t ci = 0, vi = 0, occ = nr;
        for (; ci < k; ++ci) {
            if (occ < p->cap) { in[cand[ci].u] = 1; ++occ; continue; }          /* free capacity */
            if (vi >= nr || !(res[vi].f < cand[ci].f)) break;                     /* no resident worth replacing */
            in[res[vi].u] = 0; in[cand[ci].u] = 1; ++vi;
        }
        uint32_t *row = P + (size_t)s * p->W32;
        memset(row, 0, (size_t)p->W32 * 4);
        for (uint32_t u = 0; u < p->U; ++u) if (in[u]) set_bit(row, u, 1);
    }
    free(in); free(cand); free(res);
    return KVPO_OK;
}

/*
 * Reactive Scheduling (Section IV-A): a unit that is accessed while it is not in HBM is promoted, the least
 * recently used resident makes room when HBM is full. The promotion follows the miss: the miss of step s is served
 * from off-package DRAM and the unit is resident from step s+1 on. Per step: the accessed residents become most
 * recently used; the missed units, in index order and at most `cap` of them, first take free capacity, then replace
 * the residents in order of last use (ties: lower index).
 */
int kvpo_policy_reactive(const kvpo_problem *p, uint32_t init_mode, uint32_t *P)
{
    if (p && p->birth) return KVPO_ERR_ARG;       /* the policies are defined on a fixed population */
    if (!p || !P || init_mode > 1) return KVPO_ERR_ARG;
    int rc = kvpo_init_placement(p, init_mode, P);
    if (rc) return rc;
    uint8_t *in = (uint8_t *)calloc(p->U, 1);
    uint32_t *stamp = (uint32_t *)calloc(p->U, 4);        /* 0 = never used, else step of last use + 1 */
    fu_t *res = (fu_t *)malloc(sizeof(fu_t) * p->U);
    if (!in || !stamp || !res) { free(in); free(stamp); free(res); return KVPO_ERR_NOMEM; }
    for (uint32_t u = 0; u < p->U; ++u) in[u] = (uint8_t)bit_of(P, u);
    for (uint32_t s = 0; s + 1 < p->S; ++s) {                        /* row s is final; build row s+1 */
        const uint32_t *acc = p->A + (size_t)s * p->W32;
        uint32_t nr = 0, occ = 0;
        for (uint32_t u = 0; u < p->U; ++u) {
            if (in[u] && bit_of(acc, u)) stamp[u] = s + 1;
            if (in[u]) { res[nr].f = stamp[u]; res[nr].u = u; ++nr; ++occ; }
        }
        qsort(res, nr, sizeof(fu_t), by_freq_asc);                   /* least recently used first */
        uint32_t vi = 0, promoted = 0;
        const uint32_t *was = P + (size_t)s * p->W32;                /* who was resident while step s read */
        for (uint32_t u = 0; u < p->U && promoted < p->cap; ++u) {
            if (bit_of(was, u) || !bit_of(acc, u)) continue;        /* a miss is judged against row s, not against
                                                                        evictions made a moment ago */
            if (occ < p->cap) ++occ;
            else { if (vi >= nr) break; in[res[vi].u] = 0; ++vi; }
            in[u] = 1; stamp[u] = s + 1; ++promoted;
        }
        uint32_t *row = P + (size_t)(s + 1) * p->W32;
        memset(row, 0, (size_t)p->W32 * 4);
        for (uint32_t u = 0; u < p->U; ++u) if (in[u]) set_bit(row, u, 1);
    }
    free(in); free(stamp); free(res);
    return KVPO_OK;
}

/* ------------------------------------------------------------------ */
/* The paper's own annealer (Section III-B): the state is the pair (W, R) of the look-ahead policy, the objective
 * T(W, R) the total latency of the schedule that policy produces. Here the objective comes from a table
 * T[(W-1) * n_ratio + r] (W = 1..w_max, R = r / (n_ratio - 1)) filled beforehand by running the policy and the cost
 * model on every grid point. Proposal operators and their probabilities (0.4, 0.4, 0.2), the steps {+-1, +-2} of W
 * and +-0.1 of R, the Metropolis rule, p0, alpha and the 0.1% stop rule are the paper's; a proposal that leaves the
 * grid is discarded. */
#define TAG_WR 5u

typedef struct {
    uint32_t chains, levels;
    uint64_t iters, seed;
    double p0, alpha;
    uint32_t early_stop_permille, w0, r0, reserved;
} kvpo_wr_params;

typedef struct {
    uint64_t best_ticks, final_ticks, iters_done, n_accepted;
    uint32_t best_w, best_r, final_w, final_r;
} kvpo_wr_result;

static const int WR_DW[4] = { -2, -1, 1, 2 };

/* Temperature ladder: C_0 accepts the mean uphill step between grid neighbours with probability p0. */
int kvpo_wr_temps(const uint64_t *table, uint32_t w_max, uint32_t n_ratio, const kvpo_wr_params *wp, double *temps,
                  uint64_t *mean_out)
{
    if (!table || !wp || !temps || !w_max || n_ratio < 2 || !wp->levels) return KVPO_ERR_ARG;
    if (!(wp->p0 > 0.0 && wp->p0 < 1.0) || !(wp->alpha > 0.0 && wp->alpha <= 1.0)) return KVPO_ERR_ARG;
    uint64_t sum = 0, cnt = 0;
    for (uint32_t w = 1; w <= w_max; ++w)
        for (uint32_t r = 0; r < n_ratio; ++r)
            for (int op = 0; op < 3; ++op)
                for (int a = 0; a < 4; ++a)
                    for (int b = 0; b < 2; ++b) {
                        if (op == 0 && b) continue;              /* a window move has no ratio part */
                        if (op == 1 && a) continue;              /* a ratio move has no window part */
                        int64_t nw = (int64_t)w + (op != 1 ? WR_DW[a] : 0);
                        int64_t nr = (int64_t)r + (op != 0 ? (b ? 1 : -1) : 0);
                        if (nw < 1 || nw > (int64_t)w_max || nr < 0 || nr >= (int64_t)n_ratio) continue;
                        uint64_t t0 = table[(size_t)(w - 1) * n_ratio + r], t1 = table[(size_t)(nw - 1) * n_ratio + nr];
                        if (t1 > t0) { sum += t1 - t0; ++cnt; }
                    }
    uint64_t mean = cnt ? sum / cnt : 1;
    if (!mean) mean = 1;
    if (mean_out) *mean_out = mean;
    double C = -(double)mean / log(wp->p0);
    for (uint32_t j = 0; j < wp->levels; ++j) { temps[j] = C; C = C * wp->alpha; }
    return KVPO_OK;
}

int kvpo_wr_anneal(const uint64_t *table, uint32_t w_max, uint32_t n_ratio, const kvpo_wr_params *wp,
                   const uint32_t *acc_table, const uint32_t *shifts, kvpo_wr_result *results)
{
    if (!table || !wp || !acc_table || !shifts || !results || !w_max || n_ratio < 2) return KVPO_ERR_ARG;
    if (!wp->chains || !wp->levels || !wp->iters || wp->w0 < 1 || wp->w0 > w_max || wp->r0 >= n_ratio) return KVPO_ERR_ARG;
    uint64_t per_level = wp->iters / wp->levels;
    if (!per_level) per_level = 1;
    for (uint32_t c = 0; c < wp->chains; ++c) {
        uint32_t w = wp->w0, r = wp->r0;
        uint64_t cur = table[(size_t)(w - 1) * n_ratio + r];
        kvpo_wr_result res;
        memset(&res, 0, sizeof res);
        res.best_ticks = cur; res.best_w = w; res.best_r = r;
        uint64_t best_at_boundary = cur, i = 0;
        for (; i < wp->iters; ++i) {
            uint64_t lev = i / per_level;
            if (lev > wp->levels - 1) lev = wp->levels - 1;
            if (i > 0 && i % per_level == 0 && i / per_level <= wp->levels - 1) {
                if (wp->early_stop_permille &&
                    (best_at_boundary - res.best_ticks) * 1000ull < best_at_boundary * (uint64_t)wp->early_stop_permille)
                    break;
                best_at_boundary = res.best_ticks;
            }
            uint32_t x[4];
            philox(wp->seed, (uint32_t)i, (uint32_t)(i >> 32), c, TAG_WR, x);
            uint32_t sel = x[0] & 255u;
            int op = sel < 102u ? 0 : (sel < 204u ? 1 : 2);       /* window, ratio, diagonal: 0.4, 0.4, 0.2 */
            int dw = op != 1 ? WR_DW[(x[0] >> 8) & 3u] : 0;
            int dr = op != 0 ? (((x[0] >> 10) & 1u) ? 1 : -1) : 0;
            int64_t nw = (int64_t)w + dw, nr = (int64_t)r + dr;
            if (nw < 1 || nw > (int64_t)w_max || nr < 0 || nr >= (int64_t)n_ratio) continue;
            uint64_t cand = table[(size_t)(nw - 1) * n_ratio + nr];
            int accept;
            if (cand <= cur) accept = 1;
            else {
                uint64_t q = (cand - cur) >> shifts[lev];
                accept = q < TABLE_Q && x[3] < acc_table[lev * TABLE_Q + q];
            }
            if (!accept) continue;
            ++res.n_accepted;
            w = (uint32_t)nw; r = (uint32_t)nr; cur = cand;
            if (cur < res.best_ticks) { res.best_ticks = cur; res.best_w = w; res.best_r = r; }
        }
        res.iters_done = i; res.final_ticks = cur; res.final_w = w; res.final_r = r;
        results[c] = res;
    }
    return KVPO_OK;
}

/*
 * Page Granularity Scheduling (Section IV-A): placement is managed in pages of page_units consecutive units with
 * perfect foresight of the current step's accesses. Before step s a page's score is the number of its units that
 * step s reads; non-resident pages with a positive score, ranked by score (ties: lower page index), first take free
 * page slots (capacity floor(cap / page_units) pages), then the j-th remaining one replaces the j-th resident page in
 * order of rising score (ties: lower index) while that page's score is lower. Whole pages move, so the unaccessed
 * units of a page ride along. Initial placement: the first pages up to capacity.
 */
int kvpo_policy_page(const kvpo_problem *p, uint32_t page_units, uint32_t *P)
{
    if (p && p->birth) return KVPO_ERR_ARG;       /* the policies are defined on a fixed population */
    if (!p || !P || !page_units || page_units > 32 || (page_units & (page_units - 1)) || p->U % page_units)
        return KVPO_ERR_ARG;
    const uint32_t np = p->U / page_units, cap_pages = p->cap / page_units;
    uint8_t *in = (uint8_t *)calloc(np, 1);
    fu_t *cand = (fu_t *)malloc(sizeof(fu_t) * np), *res = (fu_t *)malloc(sizeof(fu_t) * np);
    if (!in || !cand || !res) { free(in); free(cand); free(res); return KVPO_ERR_NOMEM; }
    for (uint32_t g = 0; g < cap_pages; ++g) in[g] = 1;
    for (uint32_t s = 0; s < p->S; ++s) {
        uint32_t nc = 0, nr = 0;
        for (uint32_t g = 0; g < np; ++g) {
            uint32_t f = 0;
            for (uint32_t i = 0; i < page_units; ++i) f += (uint32_t)bit_of(p->A + (size_t)s * p->W32, g * page_units + i);
            if (in[g]) { res[nr].f = f; res[nr].u = g; ++nr; }
            else if (f > 0) { cand[nc].f = f; cand[nc].u = g; ++nc; }
        }
        qsort(cand, nc, sizeof(fu_t), by_freq_desc);
        qsort(res, nr, sizeof(fu_t), by_freq_asc);
        uint32_t vi = 0, occ = nr;
        for (uint32_t ci = 0; ci < nc; ++ci) {
            if (occ < cap_pages) { in[cand[ci].u] = 1; ++occ; continue; }
            if (vi >= nr || !(res[vi].f < cand[ci].f)) break;
            in[res[vi].u] = 0; in[cand[ci].u] = 1; ++vi;
        }
        uint32_t *row = P + (size_t)s * p->W32;
        memset(row, 0, (size_t)p->W32 * 4);
        for (uint32_t g = 0; g < np; ++g)
            if (in[g]) for (uint32_t i = 0; i < page_units; ++i) set_bit(row, g * page_units + i, 1);
    }
    free(in); free(cand); free(res);
    return KVPO_OK;
}

/* ------------------------------------------------------------------ */
/* Replica exchange (parallel tempering) over the temperature ladder of
 * Section III-B: instead of one chain cooling through the levels C_0 > C_1 >
 * ..., a ladder of `rungs` replicas runs side by side, replica r of a ladder
 * starting on rung r, every replica at the fixed temperature of the rung it
 * holds; every `every` moves neighbouring rungs may exchange their states
 * (here: their rung indices, the states stay with the chains). The paper has
 * no replica exchange; the rule is the standard one for Boltzmann weights
 * exp(-T/C): rungs j (hotter) and j+1 holding states of cost E_j and E_{j+1}
 * exchange with probability min(1, exp((1/C_j - 1/C_{j+1}) (E_j - E_{j+1}))).
 * With d = E_j - E_{j+1}: d <= 0 (the colder rung holds the worse state, or
 * equal) is always accepted; d > 0 is accepted with exp(-d / C_pair),
 * 1/C_pair = 1/C_{j+1} - 1/C_j, through the same quantised table as a move
 * (kvpo_accept_table of the pair temperatures; equal temperatures exchange
 * always).
 *
 * Chains first_chain .. first_chain+chains-1, chains a multiple of rungs:
 * chain c belongs to ladder c / rungs and starts on rung c % rungs (c counted
 * from 0, not from first_chain, so that a job can be split by ladders).
 * Round t = 0, 1, ...: every chain proposes moves t*every .. min((t+1)*every,
 * moves)-1 at its rung's temperature (table row = rung), then, unless the
 * budget is used up, the pairs (j, j+1) with j = t (mod 2) try to exchange,
 * lowest j first. The uniform of pair j of ladder l in round t is word 3 of
 * Philox(counter (t_lo, t_hi, l*rungs + j, 6), key seed).
 *   table, shifts  [rungs][1024], [rungs]      : move acceptance per rung
 *   xalways        [rungs-1]                   : 1 = pair (j, j+1) always exchanges
 *   xtable, xshifts [rungs-1][1024], [rungs-1] : exchange acceptance per pair
 *   results [chains]; final_rung [chains]; n_exchanged [chains] (exchanges the chain took part in)
 *   xlog: NULL or [rounds][ladders][rungs-1][3] = {E_hot, E_cold, accepted(0/1)}, pairs not tried keep accepted = 2
 *   samples: NULL or [rounds][chains][2] = {rung held during the round, state code after the round's moves}
 *            (state code = the first two words of the schedule, for instances that small)
 *   best_states: NULL or [chains][S][W32] = every chain's schedule when it reached its best_ticks
 */
#define TAG_EXCHANGE 6u

int kvpo_anneal_exchange(const kvpo_problem *p, const kvpo_anneal_params *ap, uint32_t rungs, uint64_t every,
                         const uint32_t *table, const uint32_t *shifts, const uint32_t *xalways,
                         const uint32_t *xtable, const uint32_t *xshifts, kvpo_chain_result *results,
                         uint32_t *final_rung, uint32_t *n_exchanged, uint64_t *xlog, uint64_t *samples,
                         uint32_t *best_states)
{
    if (!p || !ap || !table || !shifts || !results || !rungs || !every) return KVPO_ERR_ARG;
    if (!ap->chains || ap->chains % rungs || ap->first_chain % rungs || !ap->moves) return KVPO_ERR_ARG;
    if (rungs > 1 && (!xalways || !xtable || !xshifts)) return KVPO_ERR_ARG;
    const uint32_t C = ap->chains, ladders = C / rungs;
    size_t nw = (size_t)p->S * p->W32;
    uint32_t *P0 = (uint32_t *)malloc(nw * 4);
    chain_state *st = (chain_state *)calloc(C, sizeof *st);
    uint32_t *rung = (uint32_t *)malloc((size_t)C * 4);
    if (!P0 || !st || !rung) { free(P0); free(st); free(rung); return KVPO_ERR_NOMEM; }
    int rc = resolve_init(p, ap, P0);
    for (uint32_t i = 0; i < C && !rc; ++i) {
        rc = state_init(p, &st[i], P0);
        memset(&results[i], 0, sizeof results[i]);
        results[i].best_ticks = st[i].cur;
        results[i].best_move = UINT64_MAX;
        rung[i] = (ap->first_chain + i) % rungs;
        if (n_exchanged) n_exchanged[i] = 0;
        if (best_states && !rc) memcpy(best_states + i * nw, st[i].P, nw * 4);
    }
    uint64_t rounds = (ap->moves + every - 1) / every;
    for (uint64_t t = 0; t < rounds && !rc; ++t) {
        uint64_t m0 = t * every, m1 = m0 + every < ap->moves ? m0 + every : ap->moves;
        for (uint32_t i = 0; i < C; ++i) {
            uint32_t chain = ap->first_chain + i, lev = rung[i];
            kvpo_chain_result *r = &results[i];
            for (uint64_t m = m0; m < m1; ++m) {
                move_t mv = decode_move(p, ap, m, chain, TAG_MOVE);
                int64_t delta; int32_t d[32][5]; uint32_t last; int changed;
                if (evaluate_move(p, &st[i], &mv, &delta, d, &last, &changed)) { ++r->n_infeasible; continue; }
                int accept;
                if (delta <= 0) accept = 1;
                else {
                    uint64_t q = (uint64_t)delta >> shifts[lev];
                    accept = q < TABLE_Q && mv.w < table[(size_t)lev * TABLE_Q + q];
                }
                if (!accept) continue;
                ++r->n_accepted;
                if (!changed) continue;
                apply_move(p, &st[i], &mv, d, last, delta);
                ++r->n_changed;
                r->traj_hash = (r->traj_hash ^ m) * 0x9E3779B97F4A7C15ull + st[i].cur;
                if (st[i].cur < r->best_ticks) {
                    r->best_ticks = st[i].cur; r->best_move = m;
                    if (best_states) memcpy(best_states + i * nw, st[i].P, nw * 4);
                }
            }
            r->moves_done = m1;
            r->final_ticks = st[i].cur;
            if (samples) {
                uint64_t code = st[i].P[0];
                if (nw > 1) code |= (uint64_t)st[i].P[1] << 32;
                samples[((size_t)t * C + i) * 2] = lev;
                samples[((size_t)t * C + i) * 2 + 1] = code;
            }
        }
        if (xlog)
            for (size_t k = 0; k < (size_t)ladders * (rungs - 1); ++k) xlog[((size_t)t * ladders * (rungs - 1) + k) * 3 + 2] = 2;
        if (m1 >= ap->moves) break;                       /* no exchange after the last round */
        for (uint32_t l = 0; l < ladders; ++l) {
            uint32_t gl = ap->first_chain / rungs + l;    /* ladder index in the whole job */
            /* who holds which rung of this ladder */
            for (uint32_t j = (uint32_t)(t & 1); j + 1 < rungs; j += 2) {
                uint32_t hot = 0, cold = 0;
                for (uint32_t i = l * rungs; i < (l + 1) * rungs; ++i) {
                    if (rung[i] == j) hot = i;
                    if (rung[i] == j + 1) cold = i;
                }
                uint64_t Eh = st[hot].cur, Ec = st[cold].cur;
                int accept;
                if (Eh <= Ec || xalways[j]) accept = 1;   /* the colder rung holds the worse state (or equal) */
                else {
                    uint32_t x[4];
                    philox(ap->seed, (uint32_t)t, (uint32_t)(t >> 32), gl * rungs + j, TAG_EXCHANGE, x);
                    uint64_t q = (Eh - Ec) >> xshifts[j];
                    accept = q < TABLE_Q && x[3] < xtable[(size_t)j * TABLE_Q + q];
                }
                if (xlog) {
                    uint64_t *e = xlog + (((size_t)t * ladders + l) * (rungs - 1) + j) * 3;
                    e[0] = Eh; e[1] = Ec; e[2] = (uint64_t)accept;
                }
                if (accept) {
                    rung[hot] = j + 1; rung[cold] = j;
                    if (n_exchanged) { ++n_exchanged[hot]; ++n_exchanged[cold]; }
                }
            }
        }
    }
    for (uint32_t i = 0; i < C; ++i) {
        if (final_rung) final_rung[i] = rung[i];
        state_free(&st[i]);
    }
    free(P0); free(st); free(rung);
    return rc;
}

/* Pair temperatures of a ladder: 1/C_pair = 1/C_{j+1} - 1/C_j (temperatures below 1 tick count as 1, as in the move
 * table). always[j] = 1 where the two temperatures are equal (or the pair temperature is beyond 2^40 ticks). */
int kvpo_exchange_temps(const double *temps, uint32_t rungs, double *pair_temps, uint32_t *always)
{
    if (!temps || !rungs || (rungs > 1 && (!pair_temps || !always))) return KVPO_ERR_ARG;
    for (uint32_t j = 0; j + 1 < rungs; ++j) {
        double a = temps[j] >= 1.0 ? temps[j] : 1.0, b = temps[j + 1] >= 1.0 ? temps[j + 1] : 1.0;
        if (b > a) return KVPO_ERR_ARG;                   /* a ladder falls */
        double inv = 1.0 / b - 1.0 / a;
        if (!(inv > 0.0) || 1.0 / inv > 1099511627776.0) { always[j] = 1; pair_temps[j] = 1.0; }
        else { always[j] = 0; pair_temps[j] = 1.0 / inv; }
    }
    return KVPO_OK;
}
