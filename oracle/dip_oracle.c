/*
 * dip_oracle.c — CPU oracle for the sparse SwiGLU decode MLP of Dynamic Input
 * Pruning (DIP) and its cache-aware variant (DIP-CA), arxiv 2412.01380.
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, step-by-step restatement
 * of the method in the paper's order and notation, in fp64 arithmetic on the
 * exact stored weight values.  It shares no code with the CUDA library and is
 * called only by the tests, by the smoke check and by the benchmark's CPU
 * baseline leg.  Nothing here is blocked, fused or reordered beyond what the
 * cited equation or algorithm states.
 *
 * Weight matrices are in the paper's canonical orientation W in R^{d_out x d_in},
 * row-major (W^u, W^g in R^{d_ff x d_model}, W^d in R^{d_model x d_ff}); the
 * unit the method keeps or drops is a COLUMN W[:, i] (Eq. 4, 7, 8).
 *
 * Pins (see tests/test_oracle_*.py): silu closed forms; dense MLP against a
 * library matmul; keep ratio 1.0 == dense; brute-force and exhaustive top-k;
 * exact-rational cache-aware ranking; ordered-list LRU replay; masked
 * mat-vec == dense mat-vec on x*m; INT4 dequant against a dequantised fp32
 * matrix; a hand-worked 2x3 example.  The paper prints no worked numeric
 * example, so no function is pinned by a published value.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (see oracle/build.py).
 * OpenMP, when enabled, only distributes independent output elements; every
 * sum runs over ascending column index in one thread.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_W_F32 = 0, ORC_W_BF16 = 1, ORC_W_INT4_G128 = 2 };
enum { ORC_GROUP = 128 };

int orc_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Threads used by the parallel loops from now on (the benchmark's single-thread
 * timing leg); every sum still runs in one thread, so results do not change. */
void orc_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n >= 1)
        omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* ------------------------------------------------------------------ *
 * Stored-number decoding (formats, not method arithmetic).
 * ------------------------------------------------------------------ */

/* bfloat16 = the upper 16 bits of an IEEE binary32. */
static double bf16_to_double(uint16_t b)
{
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
static double fp16_to_double(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    double v;
    if (e == 0)
        v = ldexp((double)f, -24);               /* subnormal or zero */
    else if (e == 31)
        v = f ? NAN : INFINITY;
    else
        v = ldexp((double)(f | 0x400), e - 25);  /* (1024+f) * 2^(e-15-10) */
    return sign ? -v : v;
}

/*
 * Element W[j, i] of a stored matrix as an exact double.
 *   F32 : float  w[d_out*d_in]
 *   BF16: uint16 w[d_out*d_in]
 *   INT4: symmetric 4-bit codes with one fp16 scale per group of 128 input
 *         indices (the GPTQ-style 4-bit setting of the paper's throughput
 *         experiments, Sec. 6.2): W[j,i] = (q[j,i] - 8) * S[i/128][j],
 *         q stored two per byte along i (even i in the low nibble),
 *         S stored as [d_in/128][d_out].
 */
double orc_weight(int type, const void *w, const uint16_t *scales,
                  int d_out, int d_in, int j, int i)
{
    size_t e = (size_t)j * (size_t)d_in + (size_t)i;
    if (type == ORC_W_F32)
        return (double)((const float *)w)[e];
    if (type == ORC_W_BF16)
        return bf16_to_double(((const uint16_t *)w)[e]);
    {
        uint8_t byte = ((const uint8_t *)w)[e >> 1];
        int q = (e & 1) ? (byte >> 4) : (byte & 0xf);
        double s = fp16_to_double(scales[(size_t)(i / ORC_GROUP) * (size_t)d_out + (size_t)j]);
        return (double)(q - 8) * s;
    }
}

/* ------------------------------------------------------------------ *
 * Eq. 2: the non-linearity sigma is SiLU, silu(z) = z * sigmoid(z).
 * ------------------------------------------------------------------ */
double orc_silu(double z)
{
    return z / (1.0 + exp(-z));
}

/* Eq. 2, element-wise: h_j = u_j * silu(g_j) for given pre-activations
 * (u = W^u x, g = W^g x, dense or sparsified), in fp64. */
void orc_glu(const double *g, const double *u, int n, double *h)
{
    for (int j = 0; j < n; ++j)
        h[j] = u[j] * orc_silu(g[j]);
}

/* ------------------------------------------------------------------ *
 * Eq. 1-2: dense MLP(x) = W^d GLU(x), GLU(x) = W^u x (.) silu(W^g x).
 * Written without any mask, as the textbook two mat-vecs, the gate
 * product and the down mat-vec.  glu_out (optional) receives GLU(x).
 * ------------------------------------------------------------------ */
void orc_dense_mlp(int type,
                   const void *Wg, const uint16_t *Sg,
                   const void *Wu, const uint16_t *Su,
                   const void *Wd, const uint16_t *Sd,
                   int d_model, int d_ff,
                   const float *x, double *glu_out, double *y)
{
    double *glu = (double *)malloc(sizeof(double) * (size_t)d_ff);
    int j;
#pragma omp parallel for schedule(static)
    for (j = 0; j < d_ff; ++j) {
        double g = 0.0, u = 0.0;
        for (int i = 0; i < d_model; ++i) {
            g += orc_weight(type, Wg, Sg, d_ff, d_model, j, i) * (double)x[i];
            u += orc_weight(type, Wu, Su, d_ff, d_model, j, i) * (double)x[i];
        }
        glu[j] = u * orc_silu(g);
    }
#pragma omp parallel for schedule(static)
    for (j = 0; j < d_model; ++j) {
        double acc = 0.0;
        for (int i = 0; i < d_ff; ++i)
            acc += orc_weight(type, Wd, Sd, d_model, d_ff, j, i) * glu[i];
        y[j] = acc;
    }
    if (glu_out)
        memcpy(glu_out, glu, sizeof(double) * (size_t)d_ff);
    free(glu);
}

/* ------------------------------------------------------------------ *
 * Eq. 10 (cache-aware score), as printed, in fp64:
 *     s_i = |x_i| * (c_i + gamma * (1 - c_i)) / ||x||_inf .
 * Reported only; the ranking uses orc_rank_key below, which orders the
 * columns identically (the denominator is one positive constant per
 * token).  For x == 0 the quotient is undefined; s is then all zero.
 * ------------------------------------------------------------------ */
void orc_ca_score(const float *x, const uint8_t *c, double gamma, int d, double *s)
{
    double norm_inf = 0.0;
    for (int i = 0; i < d; ++i) {
        double a = fabs((double)x[i]);
        if (a > norm_inf)
            norm_inf = a;
    }
    for (int i = 0; i < d; ++i) {
        double ci = c ? (double)(c[i] != 0) : 1.0;
        double num = fabs((double)x[i]) * (ci + gamma * (1.0 - ci));
        s[i] = norm_inf > 0.0 ? num / norm_inf : 0.0;
    }
}

/*
 * The number that is actually ranked: the numerator of Eq. 10 evaluated in
 * binary32 with ONE round-to-nearest multiply, u = |x| * (resident ? 1 : gamma),
 * read as its unsigned bit pattern (monotone for non-negative floats; -0 and
 * +0 coincide).  gamma == 1 or "no cache" gives the DIP key |x| of Eq. 7-8.
 * The decision is taken in binary32 so that both sides of a parity test take
 * it in the same precision.
 */
uint32_t orc_rank_key(float x, int resident, float gamma)
{
    float w = resident ? 1.0f : gamma;
    volatile float u = fabsf(x) * w;   /* volatile: one rounded binary32 product */
    float uu = u;
    uint32_t bits;
    memcpy(&bits, &uu, sizeof bits);
    return bits & 0x7fffffffu;
}

/* ------------------------------------------------------------------ *
 * topK (Sec. 3.1: keep the K largest magnitudes of the current token;
 * Alg. 1: m = topK(s, k)).  Definition written out: order all columns by
 * (key descending, index ascending) and keep the first k.  The index
 * tie-break is this library's reading; the paper is silent.
 * m[d] receives 0/1; idx[k] (optional) the kept indices in ascending order.
 * Returns 0, or -1 if k is outside [0, d].
 * ------------------------------------------------------------------ */
typedef struct { uint32_t key; int32_t idx; } orc_pair;

static int cmp_key_desc_idx_asc(const void *pa, const void *pb)
{
    const orc_pair *a = (const orc_pair *)pa, *b = (const orc_pair *)pb;
    if (a->key != b->key)
        return a->key > b->key ? -1 : 1;
    return a->idx < b->idx ? -1 : (a->idx > b->idx ? 1 : 0);
}

int orc_topk_mask(const uint32_t *key, int d, int k, uint8_t *m, int32_t *idx)
{
    if (k < 0 || k > d)
        return -1;
    orc_pair *p = (orc_pair *)malloc(sizeof(orc_pair) * (size_t)(d > 0 ? d : 1));
    for (int i = 0; i < d; ++i) {
        p[i].key = key[i];
        p[i].idx = i;
    }
    qsort(p, (size_t)d, sizeof(orc_pair), cmp_key_desc_idx_asc);
    memset(m, 0, (size_t)d);
    for (int r = 0; r < k; ++r)
        m[p[r].idx] = 1;
    free(p);
    if (idx) {
        int n = 0;
        for (int i = 0; i < d; ++i)
            if (m[i])
                idx[n++] = i;
    }
    return 0;
}

/* ------------------------------------------------------------------ *
 * c^(t) = cache_update(c^(t-1), m^(t))  (Alg. 1), with the LRU policy of
 * Sec. 5.1: the resident column whose last use lies farthest in the past is
 * evicted.  State: stamp[i] = step of the last use of column i while
 * resident, -1 if not resident; *n_resident; *step (number of updates so
 * far).  capacity = cache size in columns.
 *
 * One update, for a mask with k ones:
 *   - hits are judged against c^(t-1): hits = |m AND c^(t-1)|, misses = k-hits;
 *   - columns of the current mask are never evicted during this update;
 *   - evictions = max(0, misses - free slots), at most the number of resident
 *     columns outside the mask; victims are the smallest (stamp, index);
 *   - missed columns are inserted in ascending index while room remains; the
 *     rest are used this step without becoming resident (Sec. 6.3: when the
 *     active set exceeds the cache, part of it goes straight to the processor)
 *     and are counted as bypassed;
 *   - every column of the mask that is resident afterwards carries stamp t.
 * counters[4] += {hits, misses, evictions, bypassed}.
 * ------------------------------------------------------------------ */
typedef struct { int32_t stamp; int32_t idx; } orc_victim;

static int cmp_stamp_asc_idx_asc(const void *pa, const void *pb)
{
    const orc_victim *a = (const orc_victim *)pa, *b = (const orc_victim *)pb;
    if (a->stamp != b->stamp)
        return a->stamp < b->stamp ? -1 : 1;
    return a->idx < b->idx ? -1 : (a->idx > b->idx ? 1 : 0);
}

int orc_cache_update(int32_t *stamp, int32_t *n_resident, int32_t *step,
                     int d, int capacity, const uint8_t *m, int32_t *counters)
{
    if (capacity < 0 || capacity > d)
        return -1;
    int32_t t = *step + 1;
    int k = 0, hits = 0;
    for (int i = 0; i < d; ++i)
        if (m[i]) {
            ++k;
            if (stamp[i] >= 0)
                ++hits;
        }
    int misses = k - hits;
    int free_slots = capacity - *n_resident;
    int n_evict = misses - free_slots;
    if (n_evict < 0)
        n_evict = 0;
    int evictable = *n_resident - hits;
    if (n_evict > evictable)
        n_evict = evictable;

    /* least recently used first, among resident columns outside the mask */
    orc_victim *v = (orc_victim *)malloc(sizeof(orc_victim) * (size_t)(evictable > 0 ? evictable : 1));
    int nv = 0;
    for (int i = 0; i < d; ++i)
        if (!m[i] && stamp[i] >= 0) {
            v[nv].stamp = stamp[i];
            v[nv].idx = i;
            ++nv;
        }
    qsort(v, (size_t)nv, sizeof(orc_victim), cmp_stamp_asc_idx_asc);
    for (int e = 0; e < n_evict; ++e)
        stamp[v[e].idx] = -1;
    free(v);

    int room = free_slots + n_evict;
    int inserted = 0, bypassed = 0;
    for (int i = 0; i < d; ++i) {
        if (!m[i])
            continue;
        if (stamp[i] >= 0) {
            stamp[i] = t;                 /* hit: most recently used */
        } else if (room > 0) {
            stamp[i] = t;                 /* miss, loaded into the cache */
            --room;
            ++inserted;
        } else {
            ++bypassed;                   /* miss, used without caching */
        }
    }
    *n_resident = *n_resident - n_evict + inserted;
    *step = t;
    if (counters) {
        counters[0] += hits;
        counters[1] += misses;
        counters[2] += n_evict;
        counters[3] += bypassed;
    }
    return 0;
}

/* ------------------------------------------------------------------ *
 * The same update with the LFU policy of Sec. 5.1: a counter per column
 * tracks how often it has been used (count[i] = number of updates whose
 * mask contained column i since the state was created, kept whether or not
 * the column is resident), and the most rarely used resident column is
 * evicted.  Reading taken where the paper is silent: ties in the count go
 * to the lower column index; the columns of the current mask are pinned and
 * their counters are incremented by this update.  Everything else (hits,
 * number of evictions, ascending insertion, bypass) is as in the LRU update.
 * ------------------------------------------------------------------ */
static int cmp_count_asc_idx_asc(const void *pa, const void *pb)
{
    return cmp_stamp_asc_idx_asc(pa, pb);   /* same ordering on (value, index) pairs */
}

int orc_cache_update_lfu(int32_t *stamp, int32_t *count, int32_t *n_resident, int32_t *step,
                         int d, int capacity, const uint8_t *m, int32_t *counters)
{
    if (capacity < 0 || capacity > d)
        return -1;
    int32_t t = *step + 1;
    int k = 0, hits = 0;
    for (int i = 0; i < d; ++i)
        if (m[i]) {
            ++k;
            if (stamp[i] >= 0)
                ++hits;
        }
    int misses = k - hits;
    int free_slots = capacity - *n_resident;
    int n_evict = misses - free_slots;
    if (n_evict < 0)
        n_evict = 0;
    int evictable = *n_resident - hits;
    if (n_evict > evictable)
        n_evict = evictable;

    /* least frequently used first, among resident columns outside the mask */
    orc_victim *v = (orc_victim *)malloc(sizeof(orc_victim) * (size_t)(evictable > 0 ? evictable : 1));
    int nv = 0;
    for (int i = 0; i < d; ++i)
        if (!m[i] && stamp[i] >= 0) {
            v[nv].stamp = count[i];
            v[nv].idx = i;
            ++nv;
        }
    qsort(v, (size_t)nv, sizeof(orc_victim), cmp_count_asc_idx_asc);
    for (int e = 0; e < n_evict; ++e)
        stamp[v[e].idx] = -1;
    free(v);

    int room = free_slots + n_evict;
    int inserted = 0, bypassed = 0;
    for (int i = 0; i < d; ++i) {
        if (!m[i])
            continue;
        count[i] += 1;                    /* used once more */
        if (stamp[i] >= 0) {
            stamp[i] = t;
        } else if (room > 0) {
            stamp[i] = t;
            --room;
            ++inserted;
        } else {
            ++bypassed;
        }
    }
    *n_resident = *n_resident - n_evict + inserted;
    *step = t;
    if (counters) {
        counters[0] += hits;
        counters[1] += misses;
        counters[2] += n_evict;
        counters[3] += bypassed;
    }
    return 0;
}

/* ------------------------------------------------------------------ *
 * Belady's offline policy (Sec. 5.1: with the future reads known, evict the
 * resident column whose next use lies farthest in the future).  Replays a
 * whole trace of masks m[T][d] through a cache of `capacity` columns with the
 * same conventions as above (columns of the current mask pinned, ascending
 * insertion, bypass when nothing can be evicted) and returns the hit count;
 * misses_out (optional) receives the misses.  Ties in the next use (e.g.
 * never used again) go to the lower index.
 * ------------------------------------------------------------------ */
long long orc_belady_hits(const uint8_t *m, int T, int d, int capacity, long long *misses_out)
{
    uint8_t *res = (uint8_t *)calloc((size_t)d, 1);
    int n_res = 0;
    long long hits = 0, misses = 0;
    for (int t = 0; t < T; ++t) {
        const uint8_t *mt = m + (size_t)t * (size_t)d;
        for (int i = 0; i < d; ++i) {
            if (!mt[i])
                continue;
            if (res[i]) {
                ++hits;
                continue;
            }
            ++misses;
            if (n_res < capacity) {
                res[i] = 1;
                ++n_res;
                continue;
            }
            /* victim: resident, not in the current mask, next use farthest away */
            int victim = -1;
            long long far = -1;
            for (int j = 0; j < d; ++j) {
                if (!res[j] || mt[j])
                    continue;
                long long next = (long long)T + 1;          /* never again */
                for (int u = t + 1; u < T; ++u)
                    if (m[(size_t)u * (size_t)d + (size_t)j]) {
                        next = u;
                        break;
                    }
                if (next > far) {
                    far = next;
                    victim = j;
                }
            }
            if (victim < 0)
                continue;                                   /* bypass */
            res[victim] = 0;
            res[i] = 1;
        }
    }
    free(res);
    if (misses_out)
        *misses_out = misses;
    return hits;
}

/* ------------------------------------------------------------------ *
 * Algorithm 1, DIP-CA for one linear layer:
 *     s = score(x, c, gamma);  m = topK(s, k);  c' = cache_update(c, m).
 * The masked weights W~ = W (.) m are not materialised; the mask is returned.
 * stamp == NULL means no cache: plain DIP (Eq. 7-8), key = |x|.
 * count != NULL selects the LFU update, else LRU.
 * ------------------------------------------------------------------ */
int orc_dip_ca_mask(const float *x, int d, int k, float gamma,
                    int32_t *stamp, int32_t *count, int32_t *n_resident, int32_t *step, int capacity,
                    uint8_t *m, int32_t *idx, int32_t *counters)
{
    uint32_t *key = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)(d > 0 ? d : 1));
    for (int i = 0; i < d; ++i) {
        int resident = stamp ? (stamp[i] >= 0) : 1;
        key[i] = orc_rank_key(x[i], resident, gamma);
    }
    int rc = orc_topk_mask(key, d, k, m, idx);
    free(key);
    if (rc)
        return rc;
    if (stamp && count)
        rc = orc_cache_update_lfu(stamp, count, n_resident, step, d, capacity, m, counters);
    else if (stamp)
        rc = orc_cache_update(stamp, n_resident, step, d, capacity, m, counters);
    return rc;
}

/* ------------------------------------------------------------------ *
 * Eq. 3 with column masks (Eq. 7-8): out_j = sum_{i : m_i = 1} W[j,i] v_i,
 * i ascending, fp64.  A masked column contributes nothing ("multiplied
 * with a zero", Sec. 3.2).
 * ------------------------------------------------------------------ */
void orc_masked_matvec(int type, const void *w, const uint16_t *scales,
                       int d_out, int d_in, const float *v, const uint8_t *m, double *out)
{
    int j;
#pragma omp parallel for schedule(static)
    for (j = 0; j < d_out; ++j) {
        double acc = 0.0;
        for (int i = 0; i < d_in; ++i)
            if (m[i])
                acc += orc_weight(type, w, scales, d_out, d_in, j, i) * (double)v[i];
        out[j] = acc;
    }
}

/* ------------------------------------------------------------------ *
 * One sparse MLP step for one token (Eq. 3 with the DIP masks of Eq. 7-8,
 * each mask produced by Alg. 1 when a cache is given):
 *   m_x = mask(x, k_x)            [cache of the gate/up input]
 *   g = W~g x,  u = W~u x,  h = u (.) silu(g)            (fp64)
 *   h32 = (float) h               [h is held in binary32 between the halves]
 *   m_h = mask(h32, k_h)          [cache of the down input]
 *   y = W~d h32                                           (fp64)
 * Eq. 8 ranks |GLU~(x)|, the GLU of the already sparsified gate/up.
 * Cache arguments: stamp_* == NULL disables the cache for that input;
 * count_* != NULL selects LFU for it.
 * ------------------------------------------------------------------ */
int orc_mlp_step(int type,
                 const void *Wg, const uint16_t *Sg,
                 const void *Wu, const uint16_t *Su,
                 const void *Wd, const uint16_t *Sd,
                 int d_model, int d_ff,
                 const float *x, int k_x, int k_h, float gamma,
                 int32_t *stamp_gu, int32_t *count_gu, int32_t *nres_gu, int32_t *step_gu, int cap_gu, int32_t *ctr_gu,
                 int32_t *stamp_d, int32_t *count_d, int32_t *nres_d, int32_t *step_d, int cap_d, int32_t *ctr_d,
                 uint8_t *m_x, int32_t *idx_x, float *h32, uint8_t *m_h, int32_t *idx_h, double *y)
{
    int rc = orc_dip_ca_mask(x, d_model, k_x, gamma, stamp_gu, count_gu, nres_gu, step_gu, cap_gu,
                             m_x, idx_x, ctr_gu);
    if (rc)
        return rc;
    double *g = (double *)malloc(sizeof(double) * (size_t)d_ff);
    double *u = (double *)malloc(sizeof(double) * (size_t)d_ff);
    orc_masked_matvec(type, Wg, Sg, d_ff, d_model, x, m_x, g);
    orc_masked_matvec(type, Wu, Su, d_ff, d_model, x, m_x, u);
    for (int j = 0; j < d_ff; ++j)
        h32[j] = (float)(u[j] * orc_silu(g[j]));
    free(g);
    free(u);
    rc = orc_dip_ca_mask(h32, d_ff, k_h, gamma, stamp_d, count_d, nres_d, step_d, cap_d,
                         m_h, idx_h, ctr_d);
    if (rc)
        return rc;
    orc_masked_matvec(type, Wd, Sd, d_model, d_ff, h32, m_h, y);
    return 0;
}

/* ------------------------------------------------------------------ *
 * Gate pruning and Up pruning (Sec. 3.2, Eq. 5): one of the two d_ff-sized
 * partial activations is computed densely and ranks the MLP's neurons; the
 * rows of the other first-layer matrix and the columns of W^d that belong
 * to neurons outside the top-k are zero, and the MLP is Eq. 1-2 with those
 * pruned matrices.
 *   by = 0 (Gate pruning):  p = silu(W^g x),  m = topK(|p|),
 *                           h_j = p_j * (W^u x)_j        for j in m, else 0
 *   by = 1 (Up pruning):    p = W^u x,        m = topK(|p|),
 *                           h_j = p_j * silu((W^g x)_j)  for j in m, else 0
 *   y = sum_{j in m} W^d[:, j] h_j
 * As in the DIP step, an activation that is both ranked and multiplied is
 * held in binary32: p32 = (float) p and h32 = (float) h; sums are fp64.
 * Ties of |p32| go to the lower neuron index.
 * ------------------------------------------------------------------ */
int orc_neuron_pruned_step(int type,
                           const void *Wg, const uint16_t *Sg,
                           const void *Wu, const uint16_t *Su,
                           const void *Wd, const uint16_t *Sd,
                           int d_model, int d_ff, const float *x, int k, int by,
                           float *p32, uint8_t *m, int32_t *idx, float *h32, double *y)
{
    if (by != 0 && by != 1)
        return -1;
    const void *Wp = by == 0 ? Wg : Wu;          /* the dense, ranking matrix */
    const uint16_t *Sp = by == 0 ? Sg : Su;
    const void *Wo = by == 0 ? Wu : Wg;          /* the other one, pruned by rows */
    const uint16_t *So = by == 0 ? Su : Sg;
    int j;
#pragma omp parallel for schedule(static)
    for (j = 0; j < d_ff; ++j) {
        double acc = 0.0;
        for (int i = 0; i < d_model; ++i)
            acc += orc_weight(type, Wp, Sp, d_ff, d_model, j, i) * (double)x[i];
        p32[j] = (float)(by == 0 ? orc_silu(acc) : acc);
    }
    uint32_t *key = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)d_ff);
    for (j = 0; j < d_ff; ++j)
        key[j] = orc_rank_key(p32[j], 1, 1.0f);
    int rc = orc_topk_mask(key, d_ff, k, m, idx);
    free(key);
    if (rc)
        return rc;
#pragma omp parallel for schedule(static)
    for (j = 0; j < d_ff; ++j) {
        double acc = 0.0;
        if (m[j])
            for (int i = 0; i < d_model; ++i)
                acc += orc_weight(type, Wo, So, d_ff, d_model, j, i) * (double)x[i];
        /* a pruned row gives 0: Gate pruning 0 * p, Up pruning p * silu(0) */
        h32[j] = m[j] ? (float)((double)p32[j] * (by == 0 ? acc : orc_silu(acc))) : 0.0f;
    }
    orc_masked_matvec(type, Wd, Sd, d_model, d_ff, h32, m, y);
    return 0;
}

/* ------------------------------------------------------------------ *
 * Layer chaining used by the multi-layer workloads (not in the paper, which
 * evaluates inside full models): x_next = (x + y) / rms(x + y), fp64, rounded
 * once to binary32.  An all-zero sum is passed through unchanged.
 * ------------------------------------------------------------------ */
void orc_residual_rmsnorm(const float *x, const double *y, int d, float *x_next)
{
    double ss = 0.0;
    for (int i = 0; i < d; ++i) {
        double r = (double)x[i] + y[i];
        ss += r * r;
    }
    double rms = sqrt(ss / (double)d);
    for (int i = 0; i < d; ++i) {
        double r = (double)x[i] + y[i];
        x_next[i] = (float)(rms > 0.0 ? r / rms : r);
    }
}

/* ------------------------------------------------------------------ *
 * Batched decode: the union of B per-token masks, U = OR_b m_b (the set of
 * columns a batched step has to read once).  Returns |U|.
 * ------------------------------------------------------------------ */
int orc_mask_union(const uint8_t *m, int batch, int d, uint8_t *u)
{
    int n = 0;
    for (int i = 0; i < d; ++i) {
        uint8_t any = 0;
        for (int b = 0; b < batch; ++b)
            any |= (uint8_t)(m[(size_t)b * (size_t)d + (size_t)i] != 0);
        u[i] = any;
        n += any;
    }
    return n;
}
