/*
 * NuPS oracle: a plain, slow, single-threaded CPU statement of what the
 * parameter store's sparse access path computes.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It exists to check the CUDA library; it is
 * never part of the product path, shares no code with it, and only the tests,
 * the smoke check and the benchmark's CPU-baseline leg may load it.
 *
 * What it follows (NuPS, arXiv 2104.00501):
 *   - pull / push by key, additive updates                    Section 3.1
 *   - per-key management: replicate hot keys, keep the rest
 *     in one place; one lookup decides                         Section 3.2
 *   - replicas accumulate updates locally and a periodic
 *     sparse all-reduce (sum, only touched keys) merges them   Sections 3.1.2, 3.2
 *   - hot-set choice: access frequency > factor x mean, or the
 *     k most frequent keys                                     Section 5.1
 *   - register_distribution / PrepareSample / PullSample with
 *     partial pulls                                            Section 4.3
 *   - the four sampling schemes (independent, pooled reuse,
 *     reuse with postponing, local)                            Section 4.4
 *   - the three workload steps (skip-gram negative sampling,
 *     ComplEx with AdaGrad, matrix factorization by SGD)       Section 5.1
 *
 * The paper leaves the drawing of an iid sample from pi, the shuffle, the
 * meaning of "local" on a single machine and the step formulas open; the
 * readings taken are written beside each function.
 *
 * Arithmetic: the tables are fp32 (fp64 in the build with -DORC_REAL=double) and
 * every push is an add in that type applied in item order; everything a step
 * computes between pull and push (dots, sigmoid, square roots, losses) is done in
 * fp64 and rounded to the tables' type once.
 *
 * Pins (tests marked "not gpu"): Philox known-answer vectors; exact alias mass
 * invariant and brute-force pmf on tiny tables; chi-square of sampled
 * frequencies; the paper's worked reuse example (Section 4.4); exactly-U reuse
 * inside a U*G window; postponing invariants; conservation
 * value = init + sum of pushed deltas; finite-difference gradients of the three
 * steps; AdaGrad closed form; the +-30 clamp of the scores; the mean-instead-of-sum
 * merge.  The store and step pins run against both value types.  Loss trajectories
 * have no external pin beyond those ("parity unpinned" for absolute loss values).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef unsigned __int128 u128;

/* Value type of the tables: fp32 (the default build) or fp64 (a second build of this same file with
 * -DORC_REAL=double; Table 2 of the paper implies 8-byte values for the KGE and MF tasks).  Everything a
 * step computes between pull and push is double precision in both builds; `real` is what is stored,
 * pulled, pushed and added.                                                                          */
#ifndef ORC_REAL
#define ORC_REAL float
#endif
typedef ORC_REAL real;
int orc_value_bytes(void) { return (int)sizeof(real); }

enum { ORC_OK = 0, ORC_EINVAL = -1, ORC_ENOMEM = -2, ORC_EKEY = -4, ORC_ESTATE = -5 };
enum { ORC_SINGLE = 0, ORC_REPLICATE = 1 };
enum { ORC_CONFORM = 1, ORC_BOUNDED = 2, ORC_LONGTERM = 3, ORC_NONCONFORM = 4 };

#define ORC_MAX_DISTS 64
#define ORC_MAX_HANDLES 256
#define ORC_LOCAL_PROBES 64
#define ORC_OWNER_DEFAULT 255

/* ------------------------------------------------------------------------- */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as   */
/* easy as 1, 2, 3", SC'11): ten rounds of two 32x32->64 multiplies, with    */
/* the key bumped by the Weyl constants between rounds.                      */
/* ------------------------------------------------------------------------- */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Counter layout used by every draw of the store: (index lo, index hi, stream,
 * purpose + 256 * block).  Purposes: 0 alias draw, 1 pool permutation.        */
static void philox_at(uint64_t seed, uint64_t index, uint32_t stream, uint32_t purpose,
                      uint32_t block, uint32_t out[4])
{
    uint32_t ctr[4] = { (uint32_t)index, (uint32_t)(index >> 32), stream, purpose + 256u * block };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    orc_philox4x32_10(ctr, key, out);
}

static uint64_t mulhi64(uint64_t a, uint64_t b) { return (uint64_t)(((u128)a * b) >> 64); }
static uint32_t mulhi32(uint32_t a, uint32_t b) { return (uint32_t)(((uint64_t)a * b) >> 32); }

/* ------------------------------------------------------------------------- */
/* Alias table over integer weights (the paper only says "samples iid from   */
/* pi", Section 4.4; the table is this store's way of doing so exactly).     */
/* n buckets of capacity W = sum w; item j has mass n*w[j].  Built by one    */
/* sweep: lights (mass < W) and heavies (mass >= W) are each visited in      */
/* ascending index; the current light is topped up by the current heavy; a   */
/* heavy whose remainder falls below W is the very next light.               */
/* thr[j] = mass kept by j in its own bucket, alias[j] = who fills the rest. */
/* Returns W, or 0 when n*W would not fit 64 bits / all weights are zero.    */
/* ------------------------------------------------------------------------- */
uint64_t orc_alias_build(const uint32_t* w, uint64_t n, uint64_t* thr, uint32_t* alias)
{
    u128 Wbig = 0;
    for (uint64_t j = 0; j < n; ++j) Wbig += w[j];
    if (Wbig == 0 || Wbig * n >> 64) return 0;
    uint64_t W = (uint64_t)Wbig;

    uint64_t* heavy = (uint64_t*)malloc(sizeof(uint64_t) * (n ? n : 1));
    uint64_t nh = 0;
    for (uint64_t j = 0; j < n; ++j) {
        thr[j] = W;
        alias[j] = (uint32_t)j;
        if (n * (uint64_t)w[j] >= W) heavy[nh++] = j;
    }
    uint64_t hi = 0;                           /* current heavy = heavy[hi]        */
    uint64_t res = nh ? n * (uint64_t)w[heavy[0]] : 0; /* its remaining mass      */
    int have_pending = 0;                      /* a heavy that just became light   */
    uint64_t pend_idx = 0, pend_mass = 0;
    uint64_t next_light = 0;                   /* scan position for untouched lights */
    for (;;) {
        uint64_t l, m;
        if (have_pending) {
            l = pend_idx; m = pend_mass; have_pending = 0;
        } else {
            while (next_light < n && n * (uint64_t)w[next_light] >= W) ++next_light;
            if (next_light >= n) break;
            l = next_light++; m = n * (uint64_t)w[l];
        }
        uint64_t h = heavy[hi];
        thr[l] = m;
        alias[l] = (uint32_t)h;
        res -= (W - m);
        if (res < W) {
            have_pending = 1; pend_idx = h; pend_mass = res;
            ++hi;
            if (hi >= nh) break;               /* cannot happen: total mass is exactly n*W */
            res = n * (uint64_t)w[heavy[hi]];
        }
    }
    free(heavy);
    return W;
}

/* ------------------------------------------------------------------------- */
/* Store                                                                     */
/* ------------------------------------------------------------------------- */
typedef struct {
    int used, uniform, level;
    uint32_t key_base, U, G;
    uint64_t n, W, seed;
    uint64_t* thr;
    uint32_t* alias;
    uint64_t* off;          /* per worker: next unused position of its sample stream */
} orc_dist;

typedef struct { uint32_t key; uint8_t postponed; } lt_entry;

typedef struct {
    int used, dist;
    uint64_t N, cursor;
    uint64_t* begin;        /* [R+1] output range of each worker's sub-handle       */
    uint32_t* keys;         /* [N] materialised keys (CONFORM, BOUNDED) or the       */
                            /*     candidates k0 (NON-CONFORM)                       */
    lt_entry** list;        /* LONG-TERM: per sub-handle walk list, capacity 2*size  */
    uint64_t* pos;          /* LONG-TERM: walk position per sub-handle               */
    uint64_t* tail;         /* LONG-TERM: list length per sub-handle                 */
} orc_handle;

typedef struct {
    uint64_t num_keys;
    uint32_t L, R, sync_interval;
    int with_acc, count_accesses, track_owner;
    real *val, *acc;
    int32_t* slot;          /* key -> hot slot, -1 = single                          */
    uint32_t* hot_keys;     /* slot -> key                                           */
    uint64_t H, Hcap;
    real *dval, *dacc;     /* [R][Hcap][L] unsynced updates of each worker's replica */
    uint8_t* dirty;         /* [R][Hcap] worker's replica touched since the last sync */
    int merge_mean;         /* a sync adds the mean over the touching workers        */
    uint64_t* cnt;
    uint8_t* owner;         /* ORC_OWNER_DEFAULT = never moved: owner is key mod R   */
    uint64_t steps, syncs, hot_hits, cold_hits;
    double clip_factor;     /* 0 = updates are never clipped                         */
    double clip_sum;        /* sum of the norms of the replicated-key updates that    */
    uint64_t clip_cnt;      /*   earlier steps applied, and how many there were       */
    int status;
    orc_dist dist[ORC_MAX_DISTS];
    orc_handle handle[ORC_MAX_HANDLES];
} orc_store;

void* orc_create(uint64_t num_keys, uint32_t L, uint32_t R, int with_acc, int count_accesses,
                 int track_owner, uint32_t sync_interval)
{
    if (num_keys == 0 || num_keys > 0xFFFFFFFFull || L == 0 || R == 0 || R > 254) return NULL;
    orc_store* s = (orc_store*)calloc(1, sizeof(orc_store));
    s->num_keys = num_keys; s->L = L; s->R = R; s->sync_interval = sync_interval;
    s->with_acc = with_acc; s->count_accesses = count_accesses; s->track_owner = track_owner;
    s->val = (real*)calloc(num_keys * L, sizeof(real));
    if (with_acc) s->acc = (real*)calloc(num_keys * L, sizeof(real));
    s->slot = (int32_t*)malloc(num_keys * sizeof(int32_t));
    for (uint64_t k = 0; k < num_keys; ++k) s->slot[k] = -1;
    s->cnt = (uint64_t*)calloc(num_keys, sizeof(uint64_t));
    if (track_owner) {
        s->owner = (uint8_t*)malloc(num_keys);
        memset(s->owner, ORC_OWNER_DEFAULT, num_keys);
    }
    return s;
}

static void free_handle(orc_store* s, orc_handle* h)
{
    if (!h->used) return;
    free(h->begin); free(h->keys);
    if (h->list) { for (uint32_t q = 0; q < s->R; ++q) free(h->list[q]); free(h->list); }
    free(h->pos); free(h->tail);
    memset(h, 0, sizeof(*h));
}

void orc_destroy(void* p)
{
    orc_store* s = (orc_store*)p;
    if (!s) return;
    for (int i = 0; i < ORC_MAX_HANDLES; ++i) free_handle(s, &s->handle[i]);
    for (int i = 0; i < ORC_MAX_DISTS; ++i) { free(s->dist[i].thr); free(s->dist[i].alias); free(s->dist[i].off); }
    free(s->val); free(s->acc); free(s->slot); free(s->hot_keys); free(s->dval); free(s->dacc);
    free(s->dirty); free(s->cnt); free(s->owner); free(s);
}

real* orc_table(void* p, int which) { orc_store* s = (orc_store*)p; return which ? s->acc : s->val; }
uint64_t* orc_counts(void* p) { return ((orc_store*)p)->cnt; }
int orc_status(void* p) { orc_store* s = (orc_store*)p; int r = s->status; s->status = 0; return r; }
uint64_t orc_num_hot(void* p) { return ((orc_store*)p)->H; }
const uint32_t* orc_hot_keys(void* p) { return ((orc_store*)p)->hot_keys; }
const int32_t* orc_slots(void* p) { return ((orc_store*)p)->slot; }
void orc_stats(void* p, uint64_t out[4])
{
    orc_store* s = (orc_store*)p;
    out[0] = s->steps; out[1] = s->syncs; out[2] = s->hot_hits; out[3] = s->cold_hits;
}

/* Seeded start values: element e of the table gets an integer in [-2^23, 2^23)
 * taken from a Philox block (purpose 3), times scale * 2^-23.  One exactly
 * representable integer times one constant: the same on every machine.      */
void orc_init_uniform(void* p, int which, uint64_t seed, float scale)
{
    orc_store* s = (orc_store*)p;
    real* t = which ? s->acc : s->val;
    if (!t) return;
    float unit = scale * (1.0f / 8388608.0f);
    uint64_t total = s->num_keys * s->L;
    for (uint64_t e = 0; e < total; ++e) {
        uint32_t x[4];
        philox_at(seed, e >> 2, (uint32_t)which, 3, 0, x);
        int32_t v = (int32_t)(x[e & 3] >> 8) - 8388608;
        t[e] = (real)((float)v * unit);
    }
}

/* Worker of item i in a call over n items: contiguous chunks, q = floor(i*R/n). */
static uint32_t worker_of(const orc_store* s, uint64_t i, uint64_t n)
{
    return (uint32_t)(((u128)i * s->R) / n);
}

static int key_ok(orc_store* s, uint32_t k)
{
    if (k < s->num_keys) return 1;
    s->status = ORC_EKEY;         /* the access is skipped, the error is remembered */
    return 0;
}

static void count_one(orc_store* s, uint32_t k) { if (s->count_accesses) s->cnt[k]++; }

/* pull (Section 3.1; replicas read through the worker's own copy, Section 3.2):
 * the value at the last sync plus this worker's own unsynced updates.        */
static void pull_row(orc_store* s, uint32_t q, uint32_t k, int which, real* out)
{
    const real* t = which ? s->acc : s->val;
    const real* row = t + (uint64_t)k * s->L;
    int32_t sl = s->slot[k];
    if (sl < 0) {
        memcpy(out, row, s->L * sizeof(real));
    } else {
        const real* d = (which ? s->dacc : s->dval) + ((uint64_t)q * s->Hcap + (uint64_t)sl) * s->L;
        for (uint32_t e = 0; e < s->L; ++e) out[e] = row[e] + d[e];
    }
}

/* push (Sections 3.1, 3.1.2): additive.  A replicated key's update stays in
 * the pushing worker's replica until the next sync; any other key is updated
 * in place.                                                                 */
static void push_row(orc_store* s, uint32_t q, uint32_t k, int which, const real* d)
{
    int32_t sl = s->slot[k];
    real* dst;
    if (sl < 0) dst = (which ? s->acc : s->val) + (uint64_t)k * s->L;
    else {
        dst = (which ? s->dacc : s->dval) + ((uint64_t)q * s->Hcap + (uint64_t)sl) * s->L;
        s->dirty[(uint64_t)q * s->Hcap + (uint64_t)sl] = 1;
    }
    for (uint32_t e = 0; e < s->L; ++e) dst[e] += d[e];
}

static void note_hit(orc_store* s, uint32_t k) { if (s->slot[k] >= 0) s->hot_hits++; else s->cold_hits++; }

int orc_pull2(void* p, const uint32_t* keys, uint64_t n, real* out_val, real* out_acc)
{
    orc_store* s = (orc_store*)p;
    if (out_acc && !s->with_acc) return ORC_EINVAL;
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t k = keys[i];
        if (!key_ok(s, k)) {
            if (out_val) memset(out_val + i * s->L, 0, s->L * sizeof(real));
            if (out_acc) memset(out_acc + i * s->L, 0, s->L * sizeof(real));
            continue;
        }
        uint32_t q = worker_of(s, i, n);
        if (out_val) pull_row(s, q, k, 0, out_val + i * s->L);
        if (out_acc) pull_row(s, q, k, 1, out_acc + i * s->L);
        count_one(s, k); note_hit(s, k);
    }
    return ORC_OK;
}
int orc_pull(void* p, const uint32_t* keys, uint64_t n, real* out) { return orc_pull2(p, keys, n, out, NULL); }

int orc_push2(void* p, const uint32_t* keys, uint64_t n, const real* d_val, const real* d_acc)
{
    orc_store* s = (orc_store*)p;
    if (d_acc && !s->with_acc) return ORC_EINVAL;
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t k = keys[i];
        if (!key_ok(s, k)) continue;
        uint32_t q = worker_of(s, i, n);
        if (d_val) push_row(s, q, k, 0, d_val + i * s->L);
        if (d_acc) push_row(s, q, k, 1, d_acc + i * s->L);
        count_one(s, k); note_hit(s, k);
    }
    return ORC_OK;
}
int orc_push(void* p, const uint32_t* keys, uint64_t n, const real* d) { return orc_push2(p, keys, n, d, NULL); }

/* sync (Section 3.2: sparse all-reduce, only updated parameters): for every
 * touched hot slot, add the workers' pending updates, worker 0 first, to the
 * stored row and clear them.                                                */
int orc_sync(void* p)
{
    orc_store* s = (orc_store*)p;
    if (s->H == 0) return ORC_OK;              /* nothing replicated: no work at all */
    for (uint64_t sl = 0; sl < s->H; ++sl) {
        uint32_t touched = 0;                  /* workers whose replica of the slot was written */
        for (uint32_t r = 0; r < s->R; ++r) touched += s->dirty[(uint64_t)r * s->Hcap + sl] != 0;
        if (!touched) continue;
        uint32_t k = s->hot_keys[sl];
        for (int which = 0; which <= (s->with_acc ? 1 : 0); ++which) {
            real* row = (which ? s->acc : s->val) + (uint64_t)k * s->L;
            real* slab = which ? s->dacc : s->dval;
            for (uint32_t e = 0; e < s->L; ++e) {
                real t = 0.0f;
                for (uint32_t r = 0; r < s->R; ++r) {
                    real* d = slab + ((uint64_t)r * s->Hcap + sl) * s->L + e;
                    t += *d; *d = 0.0f;
                }
                /* option (not in the paper; it damps the summed duplicate updates of very
                 * frequent keys): the mean over the workers that pushed, not the sum      */
                if (s->merge_mean) t = t / (real)touched;
                row[e] += t;
            }
        }
        for (uint32_t r = 0; r < s->R; ++r) s->dirty[(uint64_t)r * s->Hcap + sl] = 0;
    }
    s->syncs++;
    return ORC_OK;
}

int orc_count_accesses(void* p, const uint32_t* keys, uint64_t n)
{
    orc_store* s = (orc_store*)p;
    for (uint64_t i = 0; i < n; ++i) if (key_ok(s, keys[i])) s->cnt[keys[i]]++;
    return ORC_OK;
}

/* Hot-set choice (Section 5.1).  by_topk = 0: keys whose access count exceeds
 * `param` times the mean count over all keys of the store (strictly; compared
 * as cnt * num_keys > param * total in exact integers).  by_topk = 1: the
 * `param` most frequent keys.  Either way the list is ordered by count,
 * largest first, smaller key first among equals.                            */
static const uint64_t* g_sort_cnt;
static int cmp_hot(const void* a, const void* b)
{
    uint32_t ka = *(const uint32_t*)a, kb = *(const uint32_t*)b;
    if (g_sort_cnt[ka] != g_sort_cnt[kb]) return g_sort_cnt[ka] > g_sort_cnt[kb] ? -1 : 1;
    return ka < kb ? -1 : (ka > kb ? 1 : 0);
}
uint64_t orc_select_hot(void* p, int by_topk, uint64_t param, uint32_t* out)
{
    orc_store* s = (orc_store*)p;
    uint32_t* all = (uint32_t*)malloc(s->num_keys * sizeof(uint32_t));
    uint64_t m = 0;
    if (by_topk) {
        for (uint64_t k = 0; k < s->num_keys; ++k) all[m++] = (uint32_t)k;
    } else {
        u128 total = 0;
        for (uint64_t k = 0; k < s->num_keys; ++k) total += s->cnt[k];
        for (uint64_t k = 0; k < s->num_keys; ++k)
            if ((u128)s->cnt[k] * s->num_keys > (u128)param * total) all[m++] = (uint32_t)k;
    }
    g_sort_cnt = s->cnt;
    qsort(all, m, sizeof(uint32_t), cmp_hot);
    if (by_topk && m > param) m = param;
    memcpy(out, all, m * sizeof(uint32_t));
    free(all);
    return m;
}

/* Per-key technique (Section 3.2).  Pending replica updates are merged first.
 * REPLICATE appends each not-yet-hot key, in list order (first occurrence),
 * as a new slot.  SINGLE removes the listed keys and renumbers the survivors
 * in their old order.                                                       */
int orc_set_management(void* p, const uint32_t* keys, uint64_t n, int technique)
{
    orc_store* s = (orc_store*)p;
    if (technique != ORC_SINGLE && technique != ORC_REPLICATE) return ORC_EINVAL;
    orc_sync(s);
    if (technique == ORC_REPLICATE) {
        uint64_t add = 0;
        for (uint64_t i = 0; i < n; ++i) if (keys[i] < s->num_keys) ++add;
        uint64_t need = s->H + add;
        if (need > s->Hcap) {
            /* all pending updates are zero after the sync: a fresh slab is enough */
            uint64_t cap = need;
            free(s->dval); free(s->dacc);
            s->dval = (real*)calloc((uint64_t)s->R * cap * s->L, sizeof(real));
            s->dacc = s->with_acc ? (real*)calloc((uint64_t)s->R * cap * s->L, sizeof(real)) : NULL;
            s->hot_keys = (uint32_t*)realloc(s->hot_keys, cap * sizeof(uint32_t));
            s->dirty = (uint8_t*)realloc(s->dirty, (uint64_t)s->R * cap);
            memset(s->dirty, 0, (uint64_t)s->R * cap);
            s->Hcap = cap;
        }
        for (uint64_t i = 0; i < n; ++i) {
            uint32_t k = keys[i];
            if (!key_ok(s, k) || s->slot[k] >= 0) continue;
            s->slot[k] = (int32_t)s->H;
            s->hot_keys[s->H++] = k;
        }
    } else {
        for (uint64_t i = 0; i < n; ++i) if (key_ok(s, keys[i])) s->slot[keys[i]] = -1;
        uint64_t H2 = 0;
        for (uint64_t sl = 0; sl < s->H; ++sl) {
            uint32_t k = s->hot_keys[sl];
            if (s->slot[k] < 0) continue;
            s->slot[k] = (int32_t)H2;
            s->hot_keys[H2++] = k;
        }
        s->H = H2;
    }
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* "Local" on one machine: every non-replicated key has an owning worker,    */
/* key mod R until someone localizes it; replicated keys are local to all    */
/* (Section 3.2).  A localize asked for during a call takes effect when the  */
/* call ends (relocation is asynchronous, Section 3.1.3); requests of one    */
/* call are applied in the order they were made, so the last one wins.       */
/* ------------------------------------------------------------------------- */
typedef struct { uint32_t* key; uint8_t* q; uint64_t n, cap; } loc_queue;

static int is_local(const orc_store* s, uint32_t q, uint32_t k)
{
    if (s->slot[k] >= 0) return 1;
    if (!s->owner) return 1;                   /* ownership not tracked: all local */
    uint8_t o = s->owner[k];
    return (o == ORC_OWNER_DEFAULT ? k % s->R : o) == q;
}
static void loc_request(orc_store* s, loc_queue* lq, uint32_t q, uint32_t k)
{
    if (!s->owner) return;
    if (lq->n == lq->cap) {
        lq->cap = lq->cap ? lq->cap * 2 : 1024;
        lq->key = (uint32_t*)realloc(lq->key, lq->cap * sizeof(uint32_t));
        lq->q = (uint8_t*)realloc(lq->q, lq->cap);
    }
    lq->key[lq->n] = k; lq->q[lq->n] = (uint8_t)q; lq->n++;
}
static void loc_apply(orc_store* s, loc_queue* lq)
{
    for (uint64_t i = 0; i < lq->n; ++i)
        if (s->slot[lq->key[i]] < 0) s->owner[lq->key[i]] = lq->q[i];
    free(lq->key); free(lq->q);
    memset(lq, 0, sizeof(*lq));
}

int orc_localize(void* p, const uint32_t* keys, uint64_t n)
{
    orc_store* s = (orc_store*)p;
    loc_queue lq = {0};
    for (uint64_t i = 0; i < n; ++i)
        if (key_ok(s, keys[i])) loc_request(s, &lq, worker_of(s, i, n), keys[i]);
    loc_apply(s, &lq);
    return ORC_OK;
}
int orc_owner_of(void* p, uint32_t k)
{
    orc_store* s = (orc_store*)p;
    if (k >= s->num_keys) return -1;
    if (s->slot[k] >= 0) return -2;            /* replicated: local everywhere */
    if (!s->owner) return -3;
    return s->owner[k] == ORC_OWNER_DEFAULT ? (int)(k % s->R) : (int)s->owner[k];
}

/* ------------------------------------------------------------------------- */
/* Sampling access (Sections 4.3, 4.4)                                       */
/* ------------------------------------------------------------------------- */
int orc_register_distribution(void* p, uint32_t key_base, const uint32_t* weights, uint64_t n,
                              int level, uint32_t U, uint32_t G, uint64_t seed)
{
    orc_store* s = (orc_store*)p;
    if (n == 0 || (uint64_t)key_base + n > s->num_keys) return ORC_EINVAL;
    if (level < ORC_CONFORM || level > ORC_NONCONFORM) return ORC_EINVAL;
    if ((level == ORC_BOUNDED || level == ORC_LONGTERM) && (U == 0 || G == 0)) return ORC_EINVAL;
    if ((level == ORC_LONGTERM || level == ORC_NONCONFORM) && !s->track_owner) return ORC_ESTATE;
    int id = -1;
    for (int i = 0; i < ORC_MAX_DISTS; ++i) if (!s->dist[i].used) { id = i; break; }
    if (id < 0) return ORC_ENOMEM;
    orc_dist* d = &s->dist[id];
    memset(d, 0, sizeof(*d));
    d->key_base = key_base; d->n = n; d->level = level; d->U = U; d->G = G; d->seed = seed;
    if (weights) {
        d->thr = (uint64_t*)malloc(n * sizeof(uint64_t));
        d->alias = (uint32_t*)malloc(n * sizeof(uint32_t));
        d->W = orc_alias_build(weights, n, d->thr, d->alias);
        if (d->W == 0) { free(d->thr); free(d->alias); memset(d, 0, sizeof(*d)); return ORC_EINVAL; }
    } else d->uniform = 1;
    d->off = (uint64_t*)calloc(s->R, sizeof(uint64_t));
    d->used = 1;
    return id;
}

const uint64_t* orc_dist_thr(void* p, int dist) { return ((orc_store*)p)->dist[dist].thr; }
const uint32_t* orc_dist_alias(void* p, int dist) { return ((orc_store*)p)->dist[dist].alias; }
uint64_t orc_dist_W(void* p, int dist) { return ((orc_store*)p)->dist[dist].W; }

/* One iid draw from pi: position `pos` of worker q's stream.  The 128 random
 * bits pick a bucket and a point inside it.                                 */
static uint32_t draw_iid(const orc_dist* d, uint32_t q, uint64_t pos)
{
    uint32_t x[4];
    philox_at(d->seed, pos, q, 0, 0, x);
    uint64_t a = (uint64_t)x[0] | ((uint64_t)x[1] << 32);
    uint64_t b = (uint64_t)x[2] | ((uint64_t)x[3] << 32);
    uint64_t j = mulhi64(a, d->n);
    if (!d->uniform && !(mulhi64(b, d->W) < d->thr[j])) j = d->alias[j];
    return d->key_base + (uint32_t)j;
}

/* Pooled reuse (Section 4.4): pool p holds G iid draws; it is walked U times,
 * every time (the first included) in a fresh random order.  Position s of the
 * stream is entry sigma_{p,t}(s mod G) of pool p = s / (U*G), pass
 * t = (s mod U*G) / G.  sigma comes from a Fisher-Yates shuffle, i = G-1 .. 1,
 * swap with floor(x * (i+1) / 2^32), x the next 32-bit word of the Philox
 * stream (purpose 1, index p*U + t, four words per block).                  */
static void pool_permutation(const orc_dist* d, uint32_t q, uint64_t p, uint32_t t, uint32_t* perm)
{
    uint32_t G = d->G;
    for (uint32_t i = 0; i < G; ++i) perm[i] = i;
    uint32_t x[4];
    uint32_t drawn = 0;
    for (uint32_t i = G - 1; i >= 1; --i) {
        if ((drawn & 3) == 0) philox_at(d->seed, p * d->U + t, q, 1, drawn >> 2, x);
        uint32_t r = mulhi32(x[drawn & 3], i + 1);
        ++drawn;
        uint32_t tmp = perm[i]; perm[i] = perm[r]; perm[r] = tmp;
    }
}
typedef struct { int valid; uint32_t q, t; uint64_t p; uint32_t* perm; } perm_memo;
static uint32_t draw_reuse(const orc_dist* d, uint32_t q, uint64_t pos, perm_memo* memo)
{
    uint64_t UG = (uint64_t)d->U * d->G;
    uint64_t p = pos / UG;
    uint32_t t = (uint32_t)((pos % UG) / d->G);
    uint32_t j = (uint32_t)(pos % d->G);
    if (!memo->valid || memo->q != q || memo->p != p || memo->t != t) {   /* same pass: same order */
        pool_permutation(d, q, p, t, memo->perm);
        memo->valid = 1; memo->q = q; memo->p = p; memo->t = t;
    }
    return draw_iid(d, q, p * d->G + memo->perm[j]);
}

uint32_t orc_draw_iid(void* p, int dist, uint32_t q, uint64_t pos) { return draw_iid(&((orc_store*)p)->dist[dist], q, pos); }

/* PrepareSample(dist, N) (Section 4.3).  The N output positions are cut into R
 * contiguous sub-handles, [floor(q*N/R), floor((q+1)*N/R)) for worker q; each
 * takes the next stretch of its worker's sample stream.  The sampled keys are
 * localized to that worker (Section 4.4), except under local sampling.
 * Returns the handle (>= 0) or a negative error.                            */
int64_t orc_prepare_sample(void* p, int dist, uint64_t N)
{
    orc_store* s = (orc_store*)p;
    if (dist < 0 || dist >= ORC_MAX_DISTS || !s->dist[dist].used || N == 0) return ORC_EINVAL;
    orc_dist* d = &s->dist[dist];
    int id = -1;
    for (int i = 0; i < ORC_MAX_HANDLES; ++i) if (!s->handle[i].used) { id = i; break; }
    if (id < 0) return ORC_ENOMEM;
    orc_handle* h = &s->handle[id];
    memset(h, 0, sizeof(*h));
    h->used = 1; h->dist = dist; h->N = N;
    h->begin = (uint64_t*)malloc((s->R + 1) * sizeof(uint64_t));
    for (uint32_t q = 0; q <= s->R; ++q) h->begin[q] = (uint64_t)(((u128)q * N) / s->R);
    h->keys = (uint32_t*)malloc(N * sizeof(uint32_t));
    perm_memo memo = {0};
    memo.perm = (uint32_t*)malloc((d->G ? d->G : 1) * sizeof(uint32_t));
    loc_queue lq = {0};
    for (uint32_t q = 0; q < s->R; ++q) {
        uint64_t size = h->begin[q + 1] - h->begin[q];
        for (uint64_t i = 0; i < size; ++i) {
            uint64_t pos = d->off[q] + i;
            uint32_t k = (d->level == ORC_BOUNDED || d->level == ORC_LONGTERM)
                             ? draw_reuse(d, q, pos, &memo) : draw_iid(d, q, pos);
            h->keys[h->begin[q] + i] = k;
            if (d->level != ORC_NONCONFORM) loc_request(s, &lq, q, k);
        }
        d->off[q] += size;
    }
    free(memo.perm);
    loc_apply(s, &lq);
    if (d->level == ORC_LONGTERM) {
        h->list = (lt_entry**)calloc(s->R, sizeof(lt_entry*));
        h->pos = (uint64_t*)calloc(s->R, sizeof(uint64_t));
        h->tail = (uint64_t*)calloc(s->R, sizeof(uint64_t));
        for (uint32_t q = 0; q < s->R; ++q) {
            uint64_t size = h->begin[q + 1] - h->begin[q];
            h->list[q] = (lt_entry*)malloc((2 * size + 1) * sizeof(lt_entry));
            for (uint64_t i = 0; i < size; ++i) {
                h->list[q][i].key = h->keys[h->begin[q] + i];
                h->list[q][i].postponed = 0;
            }
            h->tail[q] = size;
        }
    }
    return id;
}

/* PullSample(handle, n) (Sections 4.3, 4.4): the next n keys of the handle, in
 * the order of its sub-handles, and (if vals is given) their values as the
 * sub-handle's worker pulls them now.
 *   independent / pooled reuse: the keys fixed at PrepareSample.
 *   reuse with postponing: walk the sub-handle's list; an entry that is not
 *     local (by the ownership at the start of this call) and was not postponed
 *     before is re-localized, moved to the end of the list and skipped; an
 *     entry that was postponed once is used wherever it is.
 *   local sampling: start from the iid candidate and take the first local key
 *     at or after it (wrapping inside the distribution's key range), the
 *     candidate itself after ORC_LOCAL_PROBES failures.                     */
int orc_pull_sample(void* p, int64_t handle, uint64_t n, uint32_t* keys_out, real* vals_out)
{
    orc_store* s = (orc_store*)p;
    if (handle < 0 || handle >= ORC_MAX_HANDLES || !s->handle[handle].used) return ORC_EINVAL;
    orc_handle* h = &s->handle[handle];
    if (n > h->N - h->cursor) return ORC_ESTATE;
    orc_dist* d = &s->dist[h->dist];
    loc_queue lq = {0};
    for (uint64_t o = 0; o < n; ++o) {
        uint64_t outpos = h->cursor + o;
        uint32_t q = 0;
        while (!(h->begin[q] <= outpos && outpos < h->begin[q + 1])) ++q;
        uint32_t k;
        if (d->level == ORC_LONGTERM) {
            for (;;) {
                lt_entry* e = &h->list[q][h->pos[q]++];
                if (e->postponed || is_local(s, q, e->key)) { k = e->key; break; }
                loc_request(s, &lq, q, e->key);
                h->list[q][h->tail[q]].key = e->key;
                h->list[q][h->tail[q]].postponed = 1;
                h->tail[q]++;
            }
        } else if (d->level == ORC_NONCONFORM) {
            uint32_t k0 = h->keys[outpos];
            k = k0;
            for (uint32_t probe = 0; probe < ORC_LOCAL_PROBES; ++probe) {
                uint32_t cand = d->key_base + (uint32_t)(((uint64_t)(k0 - d->key_base) + probe) % d->n);
                if (is_local(s, q, cand)) { k = cand; break; }
            }
        } else {
            k = h->keys[outpos];
        }
        keys_out[o] = k;
        if (vals_out) pull_row(s, q, k, 0, vals_out + o * s->L);
        count_one(s, k); note_hit(s, k);
    }
    loc_apply(s, &lq);
    h->cursor += n;
    if (h->cursor == h->N) free_handle(s, h);
    return ORC_OK;
}

/* ------------------------------------------------------------------------- */
/* Workload steps (Section 5.1 names the tasks; the formulas are the usual   */
/* ones of the cited models).  A step over a batch: draw the negatives, pull */
/* everything the batch needs (a snapshot), compute every update from the    */
/* snapshot, push all updates in item order, localize the directly accessed  */
/* keys to the item's worker, and merge replicas every sync_interval steps.  */
/* ------------------------------------------------------------------------- */
static double clamp30(double x) { return x > 30.0 ? 30.0 : (x < -30.0 ? -30.0 : x); }
static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }
static double softplus(double x) { return (x > 0 ? x : 0) + log1p(exp(-fabs(x))); }

/* Gradient-norm clipping for replicated keys (Section 5.1, "Implementation and
 * cluster": updates to replicated parameters that exceed the average norm by
 * more than 2x are clipped, in the word-vector and matrix-factorization tasks).
 * Reading: the average is the mean Euclidean norm of all updates to replicated
 * keys that EARLIER steps applied (after their own clipping), so the bound is
 * fixed while a step runs and no update of a batch depends on another one of
 * the same batch; an update row d with |d| > factor * mean becomes
 * d * (factor * mean / |d|); before any such update has been applied nothing
 * is clipped.  The step's own norms join the statistics when the step ends.   */
typedef struct { double sum; uint64_t cnt; } clip_step;

void orc_set_merge_mean(void* p, int on)
{
    ((orc_store*)p)->merge_mean = on ? 1 : 0;
}

void orc_set_clipping(void* p, double factor)
{
    orc_store* s = (orc_store*)p;
    s->clip_factor = factor > 0 ? factor : 0;
}

void orc_clip_stats(void* p, double* sum, uint64_t* cnt)
{
    orc_store* s = (orc_store*)p;
    *sum = s->clip_sum; *cnt = s->clip_cnt;
}

/* d[0..L): the update about to be pushed to key k (in double, not yet rounded) */
static void clip_update(const orc_store* s, uint32_t k, double* d, clip_step* st)
{
    if (s->clip_factor == 0 || s->slot[k] < 0) return;
    double n2 = 0;
    for (uint32_t e = 0; e < s->L; ++e) n2 += d[e] * d[e];
    double n = sqrt(n2);
    if (s->clip_cnt > 0) {
        double bound = s->clip_factor * (s->clip_sum / (double)s->clip_cnt);
        if (n > bound) {
            double f = bound / n;
            for (uint32_t e = 0; e < s->L; ++e) d[e] *= f;
            n = bound;
        }
    }
    st->sum += n; st->cnt++;
}

static void clip_end_of_step(orc_store* s, const clip_step* st)
{
    s->clip_sum += st->sum; s->clip_cnt += st->cnt;
}

static void end_of_step(orc_store* s)
{
    s->steps++;
    if (s->sync_interval && s->steps % s->sync_interval == 0) orc_sync(s);
}

/* Skip-gram with negative sampling.  Item i: centre key c, context key o (an
 * output-table key), K negatives = samples i*K .. i*K+K-1 of one handle of n*K
 * samples from `dist`.  x_j = v.u_j, g_j = sigmoid(x_j) - [j==0],
 * u_j -= lr*g_j*v, v -= lr*sum_j g_j*u_j, loss = -log sig(x_0) - sum log sig(-x_j).
 * Push order within an item: o, negatives, c.  Loss = mean over items.       */
int orc_step_sgns(void* p, const uint32_t* center, const uint32_t* context, uint64_t n,
                  int dist, uint32_t K, float lr, float* loss_out, uint32_t* neg_keys_out)
{
    orc_store* s = (orc_store*)p;
    uint32_t L = s->L;
    uint64_t per = K + 2;
    uint32_t* nk = (uint32_t*)malloc((n * K + 1) * sizeof(uint32_t));
    if (K) {
        int64_t h = orc_prepare_sample(s, dist, n * K);
        if (h < 0) { free(nk); return (int)h; }
        orc_pull_sample(s, h, n * K, nk, NULL);
    }
    if (neg_keys_out) memcpy(neg_keys_out, nk, n * K * sizeof(uint32_t));
    real* upd = (real*)calloc(n * per * L, sizeof(real));
    uint32_t* uk = (uint32_t*)malloc(n * per * sizeof(uint32_t));
    uint8_t* okv = (uint8_t*)calloc(n, 1);
    real* v = (real*)malloc(L * sizeof(real));
    real* u = (real*)malloc(L * sizeof(real));
    double* gv = (double*)malloc(L * sizeof(double));
    double* dd = (double*)malloc(L * sizeof(double));
    clip_step clip = {0, 0};
    double loss = 0;
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t q = worker_of(s, i, n);
        uint32_t* kk = uk + i * per;
        kk[0] = context[i];
        for (uint32_t j = 0; j < K; ++j) kk[1 + j] = nk[i * K + j];
        kk[K + 1] = center[i];
        int ok = 1;
        for (uint64_t j = 0; j < per; ++j) ok &= key_ok(s, kk[j]);
        if (!ok) continue;
        okv[i] = 1;
        pull_row(s, q, center[i], 0, v);
        count_one(s, center[i]); count_one(s, context[i]);
        note_hit(s, center[i]); note_hit(s, context[i]);
        for (uint32_t e = 0; e < L; ++e) gv[e] = 0;
        for (uint32_t j = 0; j <= K; ++j) {
            pull_row(s, q, kk[j], 0, u);
            double x = 0;
            for (uint32_t e = 0; e < L; ++e) x += (double)v[e] * (double)u[e];
            x = clamp30(x);
            double g = sigmoid(x) - (j == 0 ? 1.0 : 0.0);
            loss += (j == 0) ? softplus(-x) : softplus(x);
            real* du = upd + (i * per + j) * L;
            for (uint32_t e = 0; e < L; ++e) {
                dd[e] = -(double)lr * g * (double)v[e];
                gv[e] += g * (double)u[e];
            }
            clip_update(s, kk[j], dd, &clip);
            for (uint32_t e = 0; e < L; ++e) du[e] = (real)dd[e];
        }
        real* dv = upd + (i * per + K + 1) * L;
        for (uint32_t e = 0; e < L; ++e) dd[e] = -(double)lr * gv[e];
        clip_update(s, center[i], dd, &clip);
        for (uint32_t e = 0; e < L; ++e) dv[e] = (real)dd[e];
    }
    clip_end_of_step(s, &clip);
    loc_queue lq = {0};
    for (uint64_t i = 0; i < n; ++i) {
        if (!okv[i]) continue;
        uint32_t q = worker_of(s, i, n);
        for (uint64_t j = 0; j < per; ++j) {
            uint32_t k = uk[i * per + j];
            push_row(s, q, k, 0, upd + (i * per + j) * L);
            count_one(s, k); note_hit(s, k);
        }
        loc_request(s, &lq, q, context[i]);
        loc_request(s, &lq, q, center[i]);
    }
    loc_apply(s, &lq);
    if (loss_out) *loss_out = (float)(loss / (double)(n ? n : 1));
    free(nk); free(upd); free(uk); free(okv); free(v); free(u); free(gv); free(dd);
    end_of_step(s);
    return ORC_OK;
}

/* ComplEx with AdaGrad.  Rows are [re(0..d-1) | im(0..d-1)], d = L/2.
 * phi(h,r,t) = sum_i re(h_i * r_i * conj(t_i)).  Item i: triple (h,r,t) and K
 * negatives e_0..e_{K-1}; e_j replaces the head when j is even, the tail when
 * odd.  loss = softplus(-phi_pos) + sum_j softplus(phi_j).  One summed
 * gradient g per key role (h, r, t, each e_j); with (w, a) the pulled value
 * and accumulator rows: push acc += g^2, val += -lr*g / (sqrt(a + g^2) + eps).
 * Push order within an item: h, r, t, e_0 .. e_{K-1}.                       */
static void complex_grads(const real* h, const real* r, const real* t, uint32_t d, double coef,
                          double* gh, double* gr, double* gt)
{
    for (uint32_t i = 0; i < d; ++i) {
        double hr = h[i], hi = h[d + i], rr = r[i], ri = r[d + i], tr = t[i], ti = t[d + i];
        if (gh) { gh[i] += coef * (rr * tr + ri * ti); gh[d + i] += coef * (rr * ti - ri * tr); }
        if (gt) { gt[i] += coef * (hr * rr - hi * ri); gt[d + i] += coef * (hi * rr + hr * ri); }
        if (gr) { gr[i] += coef * (hr * tr + hi * ti); gr[d + i] += coef * (hr * ti - hi * tr); }
    }
}
static double complex_score(const real* h, const real* r, const real* t, uint32_t d)
{
    double phi = 0;
    for (uint32_t i = 0; i < d; ++i) {
        double hr = h[i], hi = h[d + i], rr = r[i], ri = r[d + i], tr = t[i], ti = t[d + i];
        phi += hr * rr * tr + hi * rr * ti + hr * ri * ti - hi * ri * tr;
    }
    return phi;
}
int orc_step_complex(void* p, const uint32_t* hk, const uint32_t* rk, const uint32_t* tk, uint64_t n,
                     int dist, uint32_t K, float lr, float eps, float* loss_out, uint32_t* neg_keys_out)
{
    orc_store* s = (orc_store*)p;
    if (!s->with_acc || (s->L & 1)) return ORC_EINVAL;
    uint32_t L = s->L, d = L / 2;
    uint64_t per = K + 3;
    uint32_t* nk = (uint32_t*)malloc((n * K + 1) * sizeof(uint32_t));
    if (K) {
        int64_t hd = orc_prepare_sample(s, dist, n * K);
        if (hd < 0) { free(nk); return (int)hd; }
        orc_pull_sample(s, hd, n * K, nk, NULL);
    }
    if (neg_keys_out) memcpy(neg_keys_out, nk, n * K * sizeof(uint32_t));
    real* uval = (real*)calloc(n * per * L, sizeof(real));
    real* uacc = (real*)calloc(n * per * L, sizeof(real));
    uint32_t* uk = (uint32_t*)malloc(n * per * sizeof(uint32_t));
    uint8_t* okv = (uint8_t*)calloc(n, 1);
    real* rows = (real*)malloc(per * L * sizeof(real));     /* pulled values       */
    real* arow = (real*)malloc(L * sizeof(real));           /* pulled accumulator  */
    double* g = (double*)malloc(per * L * sizeof(double));
    double loss = 0;
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t q = worker_of(s, i, n);
        uint32_t* kk = uk + i * per;
        kk[0] = hk[i]; kk[1] = rk[i]; kk[2] = tk[i];
        for (uint32_t j = 0; j < K; ++j) kk[3 + j] = nk[i * K + j];
        int ok = 1;
        for (uint64_t j = 0; j < per; ++j) ok &= key_ok(s, kk[j]);
        if (!ok) continue;
        okv[i] = 1;
        for (uint64_t j = 0; j < per; ++j) pull_row(s, q, kk[j], 0, rows + j * L);
        for (int j = 0; j < 3; ++j) { count_one(s, kk[j]); note_hit(s, kk[j]); }
        for (uint64_t e = 0; e < per * L; ++e) g[e] = 0;
        const real *H = rows, *Rr = rows + L, *T = rows + 2 * L;
        double phi = clamp30(complex_score(H, Rr, T, d));
        loss += softplus(-phi);
        complex_grads(H, Rr, T, d, sigmoid(phi) - 1.0, g, g + L, g + 2 * L);
        for (uint32_t j = 0; j < K; ++j) {
            const real* E = rows + (3 + j) * L;
            double* gE = g + (3 + j) * L;
            if ((j & 1) == 0) {
                double ph = clamp30(complex_score(E, Rr, T, d));
                loss += softplus(ph);
                complex_grads(E, Rr, T, d, sigmoid(ph), gE, g + L, g + 2 * L);
            } else {
                double ph = clamp30(complex_score(H, Rr, E, d));
                loss += softplus(ph);
                complex_grads(H, Rr, E, d, sigmoid(ph), g, g + L, gE);
            }
        }
        for (uint64_t j = 0; j < per; ++j) {
            pull_row(s, q, kk[j], 1, arow);
            real* dv = uval + (i * per + j) * L;
            real* da = uacc + (i * per + j) * L;
            for (uint32_t e = 0; e < L; ++e) {
                double ge = g[j * L + e];
                double g2 = ge * ge;
                da[e] = (real)g2;
                dv[e] = (real)(-(double)lr * ge / (sqrt((double)arow[e] + g2) + (double)eps));
            }
        }
    }
    loc_queue lq = {0};
    for (uint64_t i = 0; i < n; ++i) {
        if (!okv[i]) continue;
        uint32_t q = worker_of(s, i, n);
        for (uint64_t j = 0; j < per; ++j) {
            uint32_t k = uk[i * per + j];
            push_row(s, q, k, 0, uval + (i * per + j) * L);
            push_row(s, q, k, 1, uacc + (i * per + j) * L);
            count_one(s, k); note_hit(s, k);
        }
        loc_request(s, &lq, q, hk[i]);
        loc_request(s, &lq, q, rk[i]);
        loc_request(s, &lq, q, tk[i]);
    }
    loc_apply(s, &lq);
    if (loss_out) *loss_out = (float)(loss / (double)(n ? n : 1));
    free(nk); free(uval); free(uacc); free(uk); free(okv); free(rows); free(arow); free(g);
    end_of_step(s);
    return ORC_OK;
}

/* Matrix factorization by SGD.  Cell (row key, column key, x): e = x - w.h,
 * w += lr*(e*h - l2*w), h += lr*(e*w - l2*h), loss = mean e^2.
 * Push order within an item: row, column.                                   */
int orc_step_mf(void* p, const uint32_t* rowk, const uint32_t* colk, const float* x, uint64_t n,
                float lr, float l2, float* loss_out)
{
    orc_store* s = (orc_store*)p;
    uint32_t L = s->L;
    real* upd = (real*)calloc(n * 2 * L, sizeof(real));
    uint8_t* okv = (uint8_t*)calloc(n, 1);
    real* w = (real*)malloc(L * sizeof(real));
    real* h = (real*)malloc(L * sizeof(real));
    double* dd = (double*)malloc(L * sizeof(double));
    clip_step clip = {0, 0};
    double loss = 0;
    for (uint64_t i = 0; i < n; ++i) {
        uint32_t q = worker_of(s, i, n);
        int ok = key_ok(s, rowk[i]) & key_ok(s, colk[i]);
        if (!ok) continue;
        okv[i] = 1;
        pull_row(s, q, rowk[i], 0, w);
        pull_row(s, q, colk[i], 0, h);
        count_one(s, rowk[i]); count_one(s, colk[i]);
        note_hit(s, rowk[i]); note_hit(s, colk[i]);
        double dot = 0;
        for (uint32_t e = 0; e < L; ++e) dot += (double)w[e] * (double)h[e];
        double err = (double)x[i] - dot;
        loss += err * err;
        real* dw = upd + (i * 2) * L;
        real* dh = upd + (i * 2 + 1) * L;
        for (uint32_t e = 0; e < L; ++e) dd[e] = (double)lr * (err * (double)h[e] - (double)l2 * (double)w[e]);
        clip_update(s, rowk[i], dd, &clip);
        for (uint32_t e = 0; e < L; ++e) dw[e] = (real)dd[e];
        for (uint32_t e = 0; e < L; ++e) dd[e] = (double)lr * (err * (double)w[e] - (double)l2 * (double)h[e]);
        clip_update(s, colk[i], dd, &clip);
        for (uint32_t e = 0; e < L; ++e) dh[e] = (real)dd[e];
    }
    clip_end_of_step(s, &clip);
    loc_queue lq = {0};
    for (uint64_t i = 0; i < n; ++i) {
        if (!okv[i]) continue;
        uint32_t q = worker_of(s, i, n);
        push_row(s, q, rowk[i], 0, upd + (i * 2) * L);
        push_row(s, q, colk[i], 0, upd + (i * 2 + 1) * L);
        count_one(s, rowk[i]); count_one(s, colk[i]);
        note_hit(s, rowk[i]); note_hit(s, colk[i]);
        loc_request(s, &lq, q, rowk[i]);
        loc_request(s, &lq, q, colk[i]);
    }
    loc_apply(s, &lq);
    if (loss_out) *loss_out = (float)(loss / (double)(n ? n : 1));
    free(upd); free(okv); free(w); free(h); free(dd);
    end_of_step(s);
    return ORC_OK;
}
