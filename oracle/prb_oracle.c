/*
 * prb_oracle.c -- TEST INFRASTRUCTURE, not the product.
 *
 * A plain, slow, single-threaded CPU Prioritized Replay Buffer: a K-ary sum
 * tree over transition priorities plus struct-of-arrays transition storage.
 * It exists so that the CUDA library can be compared against something that
 * can be checked against the paper by eye.  Only the tests, the smoke check
 * and the benchmark's CPU-baseline leg may call it.  It shares no source with
 * the CUDA path.
 *
 * What each part follows (PEARL, arXiv 2311.09445):
 *   - sum tree, "a parent node stores the sum of priorities of its children":
 *     Section V-A (Replay Manager).
 *   - priority sampling, the minimum index whose prefix sum reaches a uniform
 *     target x: Eq. 1 (Section II-A); done "traversing the tree performing
 *     prefix sum from root to leaf": Section V-A.
 *   - priority update / insertion along a root-leaf path: Section V-A.
 *   - Data Storage read by sampled indices: Listing 2 (Section IV-D).
 * The paper does not define stratified targets, importance-sampling weights,
 * the exponent alpha or the random stream; those follow Schaul et al.
 * (the paper's reference for prioritized replay) and Salmon et al. (Philox),
 * in the readings listed beside each function.
 *
 * Arithmetic contract (the CUDA path must reproduce it bit for bit, except the
 * IS weights which carry a 1e-5 relative tolerance):
 *   - tree nodes are IEEE binary32; a parent is ((c0 + c1) + c2) + ... in
 *     strictly left-to-right order, each add rounded to nearest-even;
 *   - sampling targets and residuals are IEEE binary64;
 *   - no fused multiply-add anywhere (build with -ffp-contract=off).
 *
 * Pinned by tests/ (see tests/test_oracle_*.py): hand-worked 8-leaf descents,
 * flat linear-scan equivalence on exactly summable priorities, incremental
 * update == rebuild, chi-square of the sampled distribution, Philox against an
 * independent implementation and published known answers, the priority
 * transform against libm pow.  Parity unpinned: the rounding-sliver rule in
 * descend() (cnt == K) on general binary32 values has no independent
 * definition to compare with; it is exercised, not pinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_NULL (-1)
#define ORACLE_ERR_BAD_FANOUT (-2)
#define ORACLE_ERR_BAD_BATCH (-3)
#define ORACLE_ERR_TOO_MANY (-4)
#define ORACLE_ERR_BAD_ARG (-7)
#define ORACLE_ERR_OOM (-6)

#define ST_BAD_INDEX 1u
#define ST_BAD_PRIORITY 2u
#define ST_EMPTY 4u
#define ST_CLAMPED 8u
#define ST_INTERNAL 16u
#define ST_STALE 32u

#define DONE_EPISODE_START 2u   /* frame-deduplicated layout: bit 1 of a slot's done byte */

#define MAX_LEVELS 64

typedef struct oracle_prb {
    uint64_t capacity;      /* N: number of leaves */
    uint32_t fanout;        /* K */
    uint32_t depth;         /* D: levels below the root; level 0 = root, level D = leaves */
    uint64_t n_nodes[MAX_LEVELS];   /* nodes in level l (without padding) */
    uint64_t n_alloc[MAX_LEVELS];   /* padded to a multiple of K (level 0: 1) */
    float *level[MAX_LEVELS];
    /* dirty bookkeeping for update(): one flag per node and a list per level */
    uint8_t *dirty[MAX_LEVELS];
    uint64_t *dirty_list[MAX_LEVELS];
    uint64_t n_dirty[MAX_LEVELS];
    /* Data Storage, struct of arrays, slot i of a field at i * field_bytes */
    uint32_t obs_bytes, act_bytes;
    uint8_t *obs, *act, *next_obs, *done;
    float *rew;
    /* Frame-deduplicated layout (stack > 0): the obs store holds ONE frame of frame_bytes per slot, the
     * next_obs store is unused, and obs_bytes = stack * frame_bytes is the size of a rebuilt stack. */
    uint32_t stack, frame_bytes;
    uint64_t size, cursor, sample_calls;
    uint32_t status;
    float max_priority;     /* largest priority written so far; 0 = none yet */
} oracle_prb_t;

/* ------------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as   */
/* easy as 1, 2, 3", SC'11).  One round: two 32x32->64 multiplies by the     */
/* constants M0, M1; the high halves are xor-ed with the other counter words */
/* and the round key; the key is bumped by the Weyl constants W0, W1 between */
/* rounds; ten rounds.                                                       */
/* ------------------------------------------------------------------------ */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)M0 * (uint64_t)c0;
        uint64_t p1 = (uint64_t)M1 * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The uniform of stratum k in sample call `call` under `seed`:
 * key = (seed low, seed high), counter = (k, 0, call low, call high),
 * u = first output word * 2^-32, a binary64 in [0, 1).
 * (Reading: the paper fixes no random stream; this layout is this library's.) */
double oracle_stratum_uniform(uint64_t seed, uint64_t call, uint32_t k)
{
    uint32_t ctr[4] = { k, 0u, (uint32_t)call, (uint32_t)(call >> 32) };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t r[4];
    oracle_philox4x32_10(ctr, key, r);
    return (double)r[0] * (1.0 / 4294967296.0);
}

/* ------------------------------------------------------------------------ */
/* Priority transform p = (|delta| + eps)^alpha (Schaul et al., proportional */
/* prioritization; the paper's "updated priority ... produced during the     */
/* computation of the loss", Section II-A).                                  */
/*                                                                           */
/* Tree contents are compared bit for bit between CPU and GPU, and the two   */
/* sides' math-library pow differ, so the power is DEFINED here through IEEE */
/* basic operations only (+, -, *, / in binary64, each rounded once):        */
/*   y  = |delta| + eps                 (binary32 add), promoted to binary64 */
/*   y  = m * 2^E, m in (sqrt(1/2), sqrt(2)]                                 */
/*   t  = (m - 1) / (m + 1)                                                  */
/*   ln m = 2 t (1 + t^2/3 + t^4/5 + ... + t^24/25)     13 terms, Horner     */
/*   L  = E * ln2 + ln m;   z = alpha * L                                    */
/*   k  = round-half-even(z / ln2);  r = (z - k*ln2_hi) - k*ln2_lo           */
/*   exp r = sum_{n=0..14} r^n / n!                     Horner               */
/*   p  = (binary32) (exp r * 2^k)                                           */
/* Returns 0 and *p on success, 1 if the entry is invalid (non-finite delta  */
/* or non-finite result).                                                    */
/* ------------------------------------------------------------------------ */
int oracle_priority_pow(float delta, float eps, float alpha, float *p)
{
    if (!isfinite(delta)) return 1;
    float y32 = fabsf(delta) + eps;
    if (!isfinite(y32)) return 1;
    if (alpha == 0.0f) { *p = 1.0f; return 0; }
    if (y32 == 0.0f) { *p = 0.0f; return 0; }

    double y = (double)y32;                 /* every nonzero binary32 is a normal binary64 */
    uint64_t bits; memcpy(&bits, &y, 8);
    int E = (int)((bits >> 52) & 0x7FFu) - 1023;
    uint64_t mbits = (bits & 0x000FFFFFFFFFFFFFull) | 0x3FF0000000000000ull;
    double m; memcpy(&m, &mbits, 8);        /* m in [1, 2) */
    if (m > 1.4142135623730951) { m = m * 0.5; E = E + 1; }

    double t = (m - 1.0) / (m + 1.0);
    double t2 = t * t;
    double S = 1.0 / 25.0;
    for (int n = 11; n >= 0; --n) {
        double coef = 1.0 / (double)(2 * n + 1);
        S = S * t2;
        S = S + coef;
    }
    double lnm = (2.0 * t) * S;

    const double LN2 = 0.6931471805599453;            /* nearest binary64 to ln 2 */
    const double LN2_HI = 0.693147180369123816490;    /* top bits of ln 2, low 32 bits zero */
    const double LN2_LO = 1.90821492927058770002e-10; /* ln 2 - LN2_HI */
    const double INV_LN2 = 1.4426950408889634;
    double L = (double)E * LN2;
    L = L + lnm;
    double z = (double)alpha * L;
    double q = z * INV_LN2;
    if (q >= 1000.0) return 1;               /* far beyond binary32 range */
    if (q <= -1000.0) { *p = 0.0f; return 0; }
    double k = rint(q);                      /* round to nearest, ties to even */
    double r = z - k * LN2_HI;
    r = r - k * LN2_LO;

    double fact = 1.0;
    for (int n = 2; n <= 14; ++n) fact = fact * (double)n;   /* 14! exact in binary64 */
    double P = 1.0 / fact;
    for (int n = 13; n >= 0; --n) {
        fact = fact / (double)(n + 1);       /* n!, exact */
        P = P * r;
        P = P + 1.0 / fact;
    }
    uint64_t sbits = (uint64_t)((int64_t)k + 1023) << 52;   /* 2^k, k in (-1000, 1000) */
    double scale; memcpy(&scale, &sbits, 8);
    float out = (float)(P * scale);
    if (!isfinite(out)) return 1;
    *p = out;
    return 0;
}

/* ------------------------------------------------------------------------ */
/* Tree geometry                                                             */
/* ------------------------------------------------------------------------ */
static uint64_t ceil_div(uint64_t a, uint64_t b) { return (a + b - 1) / b; }

static int create_impl(oracle_prb_t **out, uint64_t capacity, uint32_t fanout,
                       uint32_t obs_bytes, uint32_t act_bytes, uint32_t stack)
{
    if (!out) return ORACLE_ERR_NULL;
    if (!(fanout == 2 || fanout == 4 || fanout == 8 || fanout == 16 || fanout == 32))
        return ORACLE_ERR_BAD_FANOUT;
    if (capacity < 1 || capacity > (1ull << 30)) return ORACLE_ERR_BAD_ARG;
    oracle_prb_t *o = (oracle_prb_t *)calloc(1, sizeof(*o));
    if (!o) return ORACLE_ERR_OOM;
    o->capacity = capacity; o->fanout = fanout;
    /* D = smallest D >= 1 with K^D >= N */
    uint32_t D = 1; uint64_t span = fanout;
    while (span < capacity) { span *= fanout; ++D; }
    o->depth = D;
    o->n_nodes[D] = capacity;
    for (int l = (int)D - 1; l >= 0; --l) o->n_nodes[l] = ceil_div(o->n_nodes[l + 1], fanout);
    for (uint32_t l = 0; l <= D; ++l) {
        o->n_alloc[l] = (l == 0) ? 1 : ceil_div(o->n_nodes[l], fanout) * fanout;
        o->level[l] = (float *)calloc(o->n_alloc[l], sizeof(float));   /* +0.0f */
        o->dirty[l] = (uint8_t *)calloc(o->n_alloc[l], 1);
        o->dirty_list[l] = (uint64_t *)malloc(o->n_alloc[l] * sizeof(uint64_t));
        if (!o->level[l] || !o->dirty[l] || !o->dirty_list[l]) return ORACLE_ERR_OOM;
    }
    o->obs_bytes = obs_bytes; o->act_bytes = act_bytes;
    o->stack = stack; o->frame_bytes = stack ? obs_bytes / stack : 0;
    /* (one frame per slot and no next_obs store when frames are deduplicated) */
    o->obs = (uint8_t *)malloc((size_t)capacity * (stack ? o->frame_bytes : obs_bytes) + 1);
    o->next_obs = (uint8_t *)malloc(stack ? 1 : (size_t)capacity * obs_bytes + 1);
    o->act = (uint8_t *)malloc((size_t)capacity * act_bytes + 1);
    o->rew = (float *)malloc((size_t)capacity * sizeof(float));
    o->done = (uint8_t *)malloc((size_t)capacity);
    if (!o->obs || !o->next_obs || !o->act || !o->rew || !o->done) return ORACLE_ERR_OOM;
    *out = o;
    return ORACLE_OK;
}

int oracle_prb_create(oracle_prb_t **out, uint64_t capacity, uint32_t fanout,
                      uint32_t obs_bytes, uint32_t act_bytes)
{
    return create_impl(out, capacity, fanout, obs_bytes, act_bytes, 0);
}

/* Frame-deduplicated Data Storage (the paper's Pong workload, Table III, has 84 x 84 observations; a
 * DQN state is a stack of the last `stack` frames, so consecutive transitions of one episode share all
 * but one frame of obs and next_obs; Section VI-C: the Data Storage traffic is what dominates).
 * Reading used here -- the paper does not describe such a layout:
 *   - every slot stores ONE frame: the newest frame of its transition's next observation;
 *   - an episode begins with a marker slot (bit 1 of its done byte set) that stores the episode's
 *     first frame and is never sampled: its leaf is 0 whatever priority is given;
 *   - consecutive slots of the ring are consecutive steps; for a sampled slot i, frame(b) is the frame
 *     of slot i - min(b, c), c being the distance back to the nearest marker (or to the oldest stored
 *     slot while the ring has not wrapped): frames "before the episode" repeat its first frame;
 *     next_obs = [frame(S-1) .. frame(0)], obs = [frame(S) .. frame(1)], oldest frame first;
 *   - an insertion also clears the leaves of the `stack` slots that follow the new cursor: once the
 *     ring has wrapped they are the oldest transitions, whose history has just been overwritten;
 *     an update that names one of them is skipped with STALE. */
int oracle_prb_create_frames(oracle_prb_t **out, uint64_t capacity, uint32_t fanout,
                             uint32_t frame_bytes, uint32_t stack, uint32_t act_bytes)
{
    if (stack < 1 || stack > 16 || frame_bytes < 1 || capacity <= stack) return ORACLE_ERR_BAD_ARG;
    return create_impl(out, capacity, fanout, frame_bytes * stack, act_bytes, stack);
}

/* frame-deduplicated layout: is slot i one of the `stack` slots that follow the cursor? */
static int history_less(const oracle_prb_t *o, uint64_t i)
{
    return o->stack && (i + o->capacity - o->cursor) % o->capacity < o->stack;
}

void oracle_prb_destroy(oracle_prb_t *o)
{
    if (!o) return;
    for (uint32_t l = 0; l <= o->depth; ++l) { free(o->level[l]); free(o->dirty[l]); free(o->dirty_list[l]); }
    free(o->obs); free(o->next_obs); free(o->act); free(o->rew); free(o->done);
    free(o);
}

/* A parent is the left-to-right binary32 sum of its K children (Section V-A:
 * "a parent node stores the sum of priorities of its children"; the order is
 * this library's, fixed so the result is reproducible). */
static float sum_children(const oracle_prb_t *o, uint32_t child_level, uint64_t parent)
{
    const float *c = o->level[child_level] + parent * o->fanout;
    float s = c[0];
    for (uint32_t j = 1; j < o->fanout; ++j) s = s + c[j];
    return s;
}

/* Recompute every internal node from the leaves: the definition of the tree. */
void oracle_prb_rebuild(oracle_prb_t *o)
{
    for (int l = (int)o->depth - 1; l >= 0; --l)
        for (uint64_t j = 0; j < o->n_nodes[l]; ++j)
            o->level[l][j] = sum_children(o, (uint32_t)l + 1, j);
}

static void mark_dirty(oracle_prb_t *o, uint32_t l, uint64_t j)
{
    if (!o->dirty[l][j]) { o->dirty[l][j] = 1; o->dirty_list[l][o->n_dirty[l]++] = j; }
}

/* After leaves were written: re-sum every ancestor of a written leaf, deepest
 * level first, so each parent is computed from final children. */
static void resum_dirty(oracle_prb_t *o)
{
    for (int l = (int)o->depth; l >= 1; --l) {
        for (uint64_t t = 0; t < o->n_dirty[l]; ++t) {
            uint64_t j = o->dirty_list[l][t];
            o->dirty[l][j] = 0;
            uint64_t parent = j / o->fanout;
            o->level[l - 1][parent] = sum_children(o, (uint32_t)l, parent);
            mark_dirty(o, (uint32_t)l - 1, parent);
        }
        o->n_dirty[l] = 0;
    }
    o->dirty[0][0] = 0; o->n_dirty[0] = 0;
}

static int valid_priority(float p) { return isfinite(p) && p >= 0.0f; }

/* Running maximum of the priorities written (Schaul et al.: a new transition enters with the     */
/* maximal priority seen so far, so that it is replayed at least once).                           */
static void note_priority(oracle_prb_t *o, float p) { if (p > o->max_priority) o->max_priority = p; }
static float default_priority(const oracle_prb_t *o) { return o->max_priority > 0.0f ? o->max_priority : 1.0f; }
float oracle_prb_max_priority(const oracle_prb_t *o) { return o ? o->max_priority : 0.0f; }

/* ------------------------------------------------------------------------ */
/* Insert (Section V-A: insertion = retrieval + update; Listing 2: the new   */
/* experiences are added to the Data Storage and insertion requests sent).   */
/* Ring write at cursor .. cursor+n-1 (mod N).  The caller supplies the      */
/* priority of each new transition (the paper is silent on its value), or    */
/* passes prio = NULL: then every new transition gets the largest priority   */
/* written so far (1 if none), as in Schaul et al.  An invalid priority      */
/* (NaN, Inf, negative) stores the transition with leaf 0 and raises         */
/* BAD_PRIORITY.                                                             */
/* ------------------------------------------------------------------------ */
int oracle_prb_insert(oracle_prb_t *o, uint32_t n, const void *obs, const void *act,
                      const float *rew, const void *next_obs, const uint8_t *done,
                      const float *prio)
{
    if (!o) return ORACLE_ERR_NULL;
    if (n == 0) return ORACLE_ERR_BAD_BATCH;
    if (n > o->capacity) return ORACLE_ERR_TOO_MANY;
    if (o->stack && (next_obs || !done)) return ORACLE_ERR_BAD_ARG;   /* one frame per transition, in `obs`; markers live in `done` */
    uint32_t D = o->depth;
    const float dflt = default_priority(o);
    const uint32_t row = o->stack ? o->frame_bytes : o->obs_bytes;
    for (uint32_t t = 0; t < n; ++t) {
        uint64_t slot = (o->cursor + t) % o->capacity;
        if (obs) memcpy(o->obs + slot * row, (const uint8_t *)obs + (size_t)t * row, row);
        if (next_obs) memcpy(o->next_obs + slot * o->obs_bytes, (const uint8_t *)next_obs + (size_t)t * o->obs_bytes, o->obs_bytes);
        if (act) memcpy(o->act + slot * o->act_bytes, (const uint8_t *)act + (size_t)t * o->act_bytes, o->act_bytes);
        if (rew) o->rew[slot] = rew[t];
        if (done) o->done[slot] = done[t];
        float p = prio ? prio[t] : dflt;
        if (o->stack && (done[t] & DONE_EPISODE_START)) p = 0.0f;        /* a marker is never sampled */
        else if (!valid_priority(p)) { p = 0.0f; o->status |= ST_BAD_PRIORITY; }
        else note_priority(o, p);
        o->level[D][slot] = p;
        mark_dirty(o, D, slot);
    }
    if (o->stack) {
        /* the slots that follow the new cursor lose their history to this insertion */
        uint64_t z = o->capacity - n < o->stack ? o->capacity - n : o->stack;
        for (uint64_t s2 = 0; s2 < z; ++s2) {
            uint64_t slot = (o->cursor + n + s2) % o->capacity;
            o->level[D][slot] = 0.0f;
            mark_dirty(o, D, slot);
        }
    }
    resum_dirty(o);
    o->cursor = (o->cursor + n) % o->capacity;
    o->size = (o->size + n > o->capacity) ? o->capacity : o->size + n;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Update (Section V-A, "priority update").  The paper adds a change Delta   */
/* along the path under a mutex; in binary32 that depends on the order of    */
/* arrival.  Reading used here: SET the leaf, entries taken in batch order   */
/* (so the last valid writer of an index wins), then re-sum the ancestors.   */
/* The final tree is a function of the final leaves only.                    */
/* ------------------------------------------------------------------------ */
int oracle_prb_update_priorities(oracle_prb_t *o, uint32_t B, const int32_t *idx, const float *prio)
{
    if (!o || !idx || !prio) return ORACLE_ERR_NULL;
    if (B == 0) return ORACLE_ERR_BAD_BATCH;
    uint32_t D = o->depth;
    for (uint32_t b = 0; b < B; ++b) {
        if (idx[b] < 0 || (uint64_t)idx[b] >= o->size) { o->status |= ST_BAD_INDEX; continue; }
        if (history_less(o, (uint64_t)idx[b])) { o->status |= ST_STALE; continue; }
        if (!valid_priority(prio[b])) { o->status |= ST_BAD_PRIORITY; continue; }
        note_priority(o, prio[b]);
        o->level[D][idx[b]] = prio[b];
        mark_dirty(o, D, (uint64_t)idx[b]);
    }
    resum_dirty(o);
    return ORACLE_OK;
}

/* The paper's own form of the priority update (Section V-A, "priority update": the inputs are   */
/* indices and the change Delta of each priority).  Entry by entry, in batch order: the leaf      */
/* becomes leaf + Delta, one binary32 addition; an entry whose Delta is not finite, or whose sum   */
/* is not a valid priority (negative, not finite), is skipped with BAD_PRIORITY and leaves the     */
/* leaf as it was.  Repeated indices therefore accumulate in batch order.  Where the paper adds    */
/* Delta to every node of the root-leaf path, the ancestors here are re-summed from their          */
/* children afterwards, like after any other write: the same tree up to rounding, with every        */
/* parent still equal to the sum of its children.                                                   */
int oracle_prb_update_delta(oracle_prb_t *o, uint32_t B, const int32_t *idx, const float *delta)
{
    if (!o || !idx || !delta) return ORACLE_ERR_NULL;
    if (B == 0) return ORACLE_ERR_BAD_BATCH;
    uint32_t D = o->depth;
    for (uint32_t b = 0; b < B; ++b) {
        if (idx[b] < 0 || (uint64_t)idx[b] >= o->size) { o->status |= ST_BAD_INDEX; continue; }
        if (history_less(o, (uint64_t)idx[b])) { o->status |= ST_STALE; continue; }
        if (!isfinite(delta[b])) { o->status |= ST_BAD_PRIORITY; continue; }
        volatile float sum = o->level[D][idx[b]] + delta[b];
        float p = sum;
        if (!valid_priority(p)) { o->status |= ST_BAD_PRIORITY; continue; }
        note_priority(o, p);
        o->level[D][idx[b]] = p;
        mark_dirty(o, D, (uint64_t)idx[b]);
    }
    resum_dirty(o);
    return ORACLE_OK;
}

int oracle_prb_update(oracle_prb_t *o, uint32_t B, const int32_t *idx, const float *td,
                      float alpha, float eps)
{
    if (!o || !idx || !td) return ORACLE_ERR_NULL;
    if (B == 0) return ORACLE_ERR_BAD_BATCH;
    if (!isfinite(alpha) || alpha < 0.0f || !isfinite(eps) || eps < 0.0f) return ORACLE_ERR_BAD_ARG;
    uint32_t D = o->depth;
    for (uint32_t b = 0; b < B; ++b) {
        if (idx[b] < 0 || (uint64_t)idx[b] >= o->size) { o->status |= ST_BAD_INDEX; continue; }
        if (history_less(o, (uint64_t)idx[b])) { o->status |= ST_STALE; continue; }
        float p;
        if (oracle_priority_pow(td[b], eps, alpha, &p)) { o->status |= ST_BAD_PRIORITY; continue; }
        note_priority(o, p);
        o->level[D][idx[b]] = p;
        mark_dirty(o, D, (uint64_t)idx[b]);
    }
    resum_dirty(o);
    return ORACLE_OK;
}

/* Update that arrives after an insertion (Section IV-C, "Replay-Collision-Free Scheduling": the  */
/* insertion index is compared against the sampled indices so that the Learner's update does not */
/* contaminate a transition the Actors have written in the meantime).  `inserted` transitions    */
/* were written since the batch was sampled: they occupy the ring slots cursor-inserted ..       */
/* cursor-1 (mod capacity).  An entry that names one of them is stale: skipped, STALE raised.    */
int oracle_prb_update_after_insert(oracle_prb_t *o, uint32_t B, const int32_t *idx, const float *td,
                                   float alpha, float eps, uint32_t inserted)
{
    if (!o || !idx || !td) return ORACLE_ERR_NULL;
    if (B == 0) return ORACLE_ERR_BAD_BATCH;
    if (!isfinite(alpha) || alpha < 0.0f || !isfinite(eps) || eps < 0.0f) return ORACLE_ERR_BAD_ARG;
    if (inserted > o->capacity) return ORACLE_ERR_BAD_ARG;
    uint32_t D = o->depth;
    for (uint32_t b = 0; b < B; ++b) {
        if (idx[b] < 0 || (uint64_t)idx[b] >= o->size) { o->status |= ST_BAD_INDEX; continue; }
        /* how many slots back from the most recently written one this index lies */
        uint64_t i = (uint64_t)idx[b];
        uint64_t back = (o->cursor + o->capacity - 1 - i) % o->capacity;
        if (back < inserted || history_less(o, i)) { o->status |= ST_STALE; continue; }
        float p;
        if (oracle_priority_pow(td[b], eps, alpha, &p)) { o->status |= ST_BAD_PRIORITY; continue; }
        note_priority(o, p);
        o->level[D][idx[b]] = p;
        mark_dirty(o, D, i);
    }
    resum_dirty(o);
    return ORACLE_OK;
}

/* Priority retrieval (Section V-A): the priorities stored at the given indices.  An index outside */
/* [0, size) yields 0 and raises BAD_INDEX.                                                       */
int oracle_prb_get_priorities(oracle_prb_t *o, uint32_t B, const int32_t *idx, float *out)
{
    if (!o || !idx || !out) return ORACLE_ERR_NULL;
    if (B == 0) return ORACLE_ERR_BAD_BATCH;
    for (uint32_t b = 0; b < B; ++b) {
        if (idx[b] < 0 || (uint64_t)idx[b] >= o->size) { o->status |= ST_BAD_INDEX; out[b] = 0.0f; continue; }
        out[b] = o->level[o->depth][idx[b]];
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* One root-to-leaf traversal for target x in [0, total) (Eq. 1; Section     */
/* V-A).  At each level the K children of the current node are read, their   */
/* inclusive prefix sums s_j formed left to right in binary32 (so s_{K-1} is */
/* the parent's stored value), and the first child with x < s_j is taken;    */
/* the residual x - s_{j-1} is carried down in binary64.                     */
/*                                                                           */
/* Reading of Eq. 1: the paper writes "prefix sum >= x" with x in [0, sum];  */
/* used here are half-open intervals S_{i-1} <= x < S_i with x in [0, sum),  */
/* the same distribution, which never selects a zero-priority leaf.          */
/* If rounding leaves x >= s_{K-1} (paper silent): take the last child with  */
/* a positive value and raise CLAMPED; if no child is positive take child 0  */
/* and raise INTERNAL.                                                       */
/* ------------------------------------------------------------------------ */
int64_t oracle_prb_descend(oracle_prb_t *o, double x, float *leaf_priority)
{
    uint32_t K = o->fanout;
    uint64_t g = 0;
    for (uint32_t l = 1; l <= o->depth; ++l) {
        const float *c = o->level[l] + g * K;
        float s[32];
        s[0] = c[0];
        for (uint32_t j = 1; j < K; ++j) s[j] = s[j - 1] + c[j];
        uint32_t cnt = 0;
        for (uint32_t j = 0; j < K; ++j) if (x >= (double)s[j]) ++cnt;
        uint32_t j;
        if (cnt < K) {
            j = cnt;
        } else {
            o->status |= ST_CLAMPED;
            int last = -1;
            for (uint32_t i = 0; i < K; ++i) if (c[i] > 0.0f) last = (int)i;
            if (last < 0) { o->status |= ST_INTERNAL; last = 0; }
            j = (uint32_t)last;
        }
        if (j > 0) x = x - (double)s[j - 1];
        g = g * K + j;
    }
    if (leaf_priority) *leaf_priority = o->level[o->depth][g];
    return (int64_t)g;
}

/* Stratified targets (Schaul et al.: the range [0, total) is cut into B equal
 * segments and one value drawn uniformly from each):
 *   x_k = (k + u_k) * (total / B), binary64, clamped below total. */
void oracle_prb_targets(oracle_prb_t *o, uint32_t B, uint64_t seed, uint64_t call, double *x)
{
    double total = (double)o->level[0][0];
    double seg = total / (double)B;
    for (uint32_t k = 0; k < B; ++k) {
        double u = oracle_stratum_uniform(seed, call, k);
        double xk = ((double)k + u) * seg;
        if (xk >= total) xk = nextafter(total, 0.0);
        x[k] = xk;
    }
}

/* The observations of slot i into obs / next_obs (either may be NULL): the stored rows, or, with the
 * frame-deduplicated layout, the two stacks rebuilt from consecutive slots (see oracle_prb_create_frames). */
static void copy_observations(const oracle_prb_t *o, uint64_t i, uint8_t *obs, uint8_t *next_obs)
{
    if (!o->stack) {
        if (obs) memcpy(obs, o->obs + i * o->obs_bytes, o->obs_bytes);
        if (next_obs) memcpy(next_obs, o->next_obs + i * o->obs_bytes, o->obs_bytes);
        return;
    }
    const uint32_t S = o->stack, F = o->frame_bytes;
    /* c: how far back frames may be taken -- to the nearest marker, or to slot 0 while the ring has not wrapped */
    uint32_t c = S;
    for (uint32_t d = 1; d <= S; ++d) {
        if (o->size < o->capacity && i < d) { c = d - 1; break; }        /* nothing is stored before slot 0 */
        uint64_t j = (i + o->capacity - d) % o->capacity;
        if (o->done[j] & DONE_EPISODE_START) { c = d; break; }
    }
    for (uint32_t pos = 0; pos < S; ++pos) {          /* pos 0 = oldest frame of a stack */
        uint32_t b_next = S - 1 - pos, b_obs = S - pos;                  /* distances back from slot i */
        uint64_t j_next = (i + o->capacity - (b_next < c ? b_next : c)) % o->capacity;
        uint64_t j_obs = (i + o->capacity - (b_obs < c ? b_obs : c)) % o->capacity;
        if (next_obs) memcpy(next_obs + (size_t)pos * F, o->obs + j_next * F, F);
        if (obs) memcpy(obs + (size_t)pos * F, o->obs + j_obs * F, F);
    }
}

/* ------------------------------------------------------------------------ */
/* Sample B transitions: indices (Eq. 1 per stratum), importance-sampling    */
/* weights and the gathered batch (Listing 2: sampled_data =                 */
/* D_storage[sampled_indices]).                                              */
/*   P(i) = p_i / total;  w_i = (size * P(i))^(-beta) / max_j w_j            */
/* (Schaul et al.; "size" = transitions currently stored; the maximum runs   */
/* over this batch).  Weights are formed in binary64 and rounded to binary32.*/
/* Any output pointer except idx may be NULL.  An empty buffer or a          */
/* non-positive total raises EMPTY and leaves outputs and the call counter   */
/* untouched.                                                                */
/* ------------------------------------------------------------------------ */
static int sample_impl(oracle_prb_t *o, uint32_t B, float beta, uint64_t seed,
                       int32_t *idx, float *w, void *obs, void *act, float *rew,
                       void *next_obs, uint8_t *done, int buffer_norm)
{
    if (!o || !idx) return ORACLE_ERR_NULL;
    if (B == 0) return ORACLE_ERR_BAD_BATCH;
    if (!isfinite(beta) || beta < 0.0f) return ORACLE_ERR_BAD_ARG;
    float total32 = o->level[0][0];
    if (o->size == 0 || !(total32 > 0.0f)) { o->status |= ST_EMPTY; return ORACLE_OK; }
    double total = (double)total32;
    double *x = (double *)malloc((size_t)B * sizeof(double));
    double *wraw = (double *)malloc((size_t)B * sizeof(double));
    if (!x || !wraw) { free(x); free(wraw); return ORACLE_ERR_OOM; }
    oracle_prb_targets(o, B, seed, o->sample_calls, x);
    double wmax = 0.0;
    for (uint32_t k = 0; k < B; ++k) {
        float p;
        int64_t i = oracle_prb_descend(o, x[k], &p);
        idx[k] = (int32_t)i;
        double prob_times_size = (double)o->size * (double)p / total;
        wraw[k] = pow(prob_times_size, -(double)beta);
        if (wraw[k] > wmax) wmax = wraw[k];
    }
    if (buffer_norm) {
        /* the largest weight any stored transition could get: that of the smallest positive priority */
        float pmin = 0.0f;
        for (uint64_t i = 0; i < o->size; ++i) {
            float p = o->level[o->depth][i];
            if (p > 0.0f && (pmin == 0.0f || p < pmin)) pmin = p;
        }
        wmax = pow((double)o->size * (double)pmin / total, -(double)beta);
    }
    if (w) for (uint32_t k = 0; k < B; ++k) w[k] = (float)(wraw[k] / wmax);
    for (uint32_t k = 0; k < B; ++k) {
        uint64_t i = (uint64_t)idx[k];
        copy_observations(o, i, obs ? (uint8_t *)obs + (size_t)k * o->obs_bytes : NULL,
                          next_obs ? (uint8_t *)next_obs + (size_t)k * o->obs_bytes : NULL);
        if (act) memcpy((uint8_t *)act + (size_t)k * o->act_bytes, o->act + i * o->act_bytes, o->act_bytes);
        if (rew) rew[k] = o->rew[i];
        if (done) done[k] = o->done[i];
    }
    free(x); free(wraw);
    o->sample_calls += 1;
    return ORACLE_OK;
}

int oracle_prb_sample(oracle_prb_t *o, uint32_t B, float beta, uint64_t seed,
                      int32_t *idx, float *w, void *obs, void *act, float *rew,
                      void *next_obs, uint8_t *done)
{
    return sample_impl(o, B, beta, seed, idx, w, obs, act, rew, next_obs, done, 0);
}

/* The same sample with the weights normalised as in the prioritized-replay paper the toolkit    */
/* follows (Schaul et al., Algorithm 1: w_j = (N P(j))^-beta / max_i w_i with the maximum over the */
/* whole memory): the divisor is the weight of the smallest positive priority in the buffer,     */
/* (N p_min / total)^-beta, found by a plain scan.  Weights are then at most 1 and do not depend   */
/* on which other transitions the batch happens to hold.                                           */
int oracle_prb_sample_buffer_norm(oracle_prb_t *o, uint32_t B, float beta, uint64_t seed,
                                  int32_t *idx, float *w, void *obs, void *act, float *rew,
                                  void *next_obs, uint8_t *done)
{
    return sample_impl(o, B, beta, seed, idx, w, obs, act, rew, next_obs, done, 1);
}

int oracle_prb_read_rows(oracle_prb_t *o, const int32_t *idx, uint32_t n, void *obs, void *act,
                         float *rew, void *next_obs, uint8_t *done);

/* Uniform replay (Section III-B: the toolkit's replay mode besides "prioritized"): B independent */
/* draws i_k = floor(u_k * size), u_k from the same Philox stream and call counter as the          */
/* prioritized sample; weights are all 1; rows are gathered as usual.                              */
int oracle_prb_sample_uniform(oracle_prb_t *o, uint32_t B, uint64_t seed, int32_t *idx, float *w, void *obs,
                              void *act, float *rew, void *next_obs, uint8_t *done)
{
    if (!o || !idx) return ORACLE_ERR_NULL;
    if (B == 0) return ORACLE_ERR_BAD_BATCH;
    if (o->stack) return ORACLE_ERR_BAD_ARG;      /* a uniform draw could name a marker or a slot without history */
    if (o->size == 0) { o->status |= ST_EMPTY; return ORACLE_OK; }
    for (uint32_t k = 0; k < B; ++k) {
        uint32_t ctr[4] = { k, 0u, (uint32_t)o->sample_calls, (uint32_t)(o->sample_calls >> 32) };
        uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
        uint32_t r[4];
        oracle_philox4x32_10(ctr, key, r);
        idx[k] = (int32_t)(((uint64_t)r[0] * o->size) >> 32);        /* floor(r0 / 2^32 * size) */
        if (w) w[k] = 1.0f;
    }
    int rc = oracle_prb_read_rows(o, idx, B, obs, act, rew, next_obs, done);
    if (rc != ORACLE_OK) return rc;
    o->sample_calls += 1;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Read-back                                                                 */
/* ------------------------------------------------------------------------ */
int oracle_prb_info(oracle_prb_t *o, uint64_t *size, uint64_t *cursor, uint64_t *sample_calls, uint32_t *depth)
{
    if (!o) return ORACLE_ERR_NULL;
    if (size) *size = o->size;
    if (cursor) *cursor = o->cursor;
    if (sample_calls) *sample_calls = o->sample_calls;
    if (depth) *depth = o->depth;
    return ORACLE_OK;
}

uint64_t oracle_prb_level_nodes(oracle_prb_t *o, uint32_t level) { return (o && level <= o->depth) ? o->n_nodes[level] : 0; }
uint64_t oracle_prb_level_alloc(oracle_prb_t *o, uint32_t level) { return (o && level <= o->depth) ? o->n_alloc[level] : 0; }

/* Copies `count` entries of level `level` (0 = root), padding included. */
int oracle_prb_read_level(oracle_prb_t *o, uint32_t level, float *dst, uint64_t count)
{
    if (!o || !dst) return ORACLE_ERR_NULL;
    if (level > o->depth || count > o->n_alloc[level]) return ORACLE_ERR_BAD_ARG;
    memcpy(dst, o->level[level], (size_t)count * sizeof(float));
    return ORACLE_OK;
}

/* Test hook: overwrite tree entries directly (used to plant mistakes and to
 * build hand-worked trees). */
int oracle_prb_poke_level(oracle_prb_t *o, uint32_t level, uint64_t first, const float *src, uint64_t count)
{
    if (!o || !src) return ORACLE_ERR_NULL;
    if (level > o->depth || first + count > o->n_alloc[level]) return ORACLE_ERR_BAD_ARG;
    memcpy(o->level[level] + first, src, (size_t)count * sizeof(float));
    return ORACLE_OK;
}

int oracle_prb_read_rows(oracle_prb_t *o, const int32_t *idx, uint32_t n, void *obs, void *act,
                         float *rew, void *next_obs, uint8_t *done)
{
    if (!o || !idx) return ORACLE_ERR_NULL;
    for (uint32_t k = 0; k < n; ++k) {
        if (idx[k] < 0 || (uint64_t)idx[k] >= o->capacity) return ORACLE_ERR_BAD_ARG;
        uint64_t i = (uint64_t)idx[k];
        copy_observations(o, i, obs ? (uint8_t *)obs + (size_t)k * o->obs_bytes : NULL,
                          next_obs ? (uint8_t *)next_obs + (size_t)k * o->obs_bytes : NULL);
        if (act) memcpy((uint8_t *)act + (size_t)k * o->act_bytes, o->act + i * o->act_bytes, o->act_bytes);
        if (rew) rew[k] = o->rew[i];
        if (done) done[k] = o->done[i];
    }
    return ORACLE_OK;
}

/* Returns the accumulated status bits and clears them. */
uint32_t oracle_prb_status(oracle_prb_t *o)
{
    if (!o) return 0;
    uint32_t s = o->status; o->status = 0; return s;
}
