/*
 * RanDeS CPU oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, element-by-element implementation of delta superposition and
 * retrieval under seed-defined random orthogonal transforms, written from the
 * paper's equations.  It exists so that the CUDA library can be compared with
 * something that can be checked against the paper by eye.  Only tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it; it shares no
 * code with the CUDA library and neither includes the other.
 *
 * Notation (paper symbol in brackets):
 *   W_0  base model            [Theta_0]
 *   W_i  fine-tuned model i    [Theta_i]
 *   d_i  = W_i - W_0           [Delta_i, Section 3]
 *   T_i  orthogonal transform  [O_i, Section 4]
 *   M    = sum_i T_i(d_i)      [the superposed delta, Section 4 / Eq. in 4.4]
 *   sigma_i^g  permutation of the members of group g for task i [Section 4.3]
 *   s_i(l,c)   +-1 diagonal entry for task i, slot l, column c   [Section 4.4]
 *
 * Readings of points the paper leaves open (all are stated again in the
 * design notes of this repository):
 *   - T_i = D_i o P_i: the layers of a delta are shuffled first, the sign flip
 *     is indexed by the position ("slot") the layer lands on in M.
 *   - Shuffle is the gather the paper prints: slot k receives member sigma(k).
 *   - lambda is applied at retrieval; M is kept in fp32 by default, whatever the
 *     storage type of the weights.  With m_dtype = bf16 (a smaller superposition,
 *     which the conclusion names as future work without fixing a format)
 *     compress sums in fp32 and rounds each element once at the end; add and
 *     remove widen the stored element, add in fp32 and round again; retrieve
 *     widens it.
 *   - "Column" is the second (contiguous) index of a row-major [rows, cols]
 *     array; a 1-D parameter is [1, cols].
 *   - Random numbers: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11),
 *     key = the task's 64-bit seed, counter = (index, layer-or-group, domain
 *     tag, task id).
 *   - Skip rate k (appendix on the dynamics between shuffling and sign flips):
 *     of the members of a group, in layer order, those with index 0, k, 2k, ...
 *     take part in the shuffle (among themselves) and in the flip; the others
 *     are left as they are.
 *   - Layer shifting (same appendix: a deterministic move of every layer
 *     to the next depth, the last wrapping to the first) is read as a rotation of the participating members towards higher block
 *     index; task t rotates by 1 + (t mod (n - 1)) positions (n participants),
 *     so that different tasks are misaligned and no task gets the identity.
 *     Slot k then receives member (k - shift) mod n.
 *   - Arithmetic: fp32; the subtraction W_i - W_0 and each accumulation are
 *     separately rounded; retrieval is one fused multiply-add; bf16 is
 *     round-to-nearest-even.
 *
 * Every function below is pinned by the CPU test-suite to something other
 * than itself (known-answer vectors, dense signed-permutation matrices in
 * double precision, closed forms, invariants).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define RO_F32 0
#define RO_BF16 1
#define RO_SHUFFLE 1u
#define RO_FLIP 2u
#define RO_SHIFT 4u                      /* deterministic rotation instead of a random permutation */
#define RO_SKIP(flags) (((flags) >> 8) & 0xFFu) /* every k-th member of a group takes part; 0 and 1 = all */

#define RO_GAUSS (1u << 16)              /* Gaussian-like diagonal context (Section 5.5, "RD") instead of the +-1 one */
#define RO_TAG_GAUS 0x47415553u /* "GAUS" */
#define RO_TAG_PERM 0x5045524Du /* "PERM" */
#define RO_TAG_SIGN 0x5349474Eu /* "SIGN" */

/* ------------------------------------------------------------------------ */
/* Philox4x32-10, from the published definition (SC'11, Section 3.3 / Table  */
/* of multipliers): ten rounds of two 32x32->64 multiplies, the key bumped   */
/* by the Weyl constants between rounds.                                     */
/* ------------------------------------------------------------------------ */
void ro_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t MUL0 = 0xD2511F53u, MUL1 = 0xCD9E8D57u;
    const uint32_t WEYL0 = 0x9E3779B9u, WEYL1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) {
            k0 += WEYL0;
            k1 += WEYL1;
        }
        uint64_t p0 = (uint64_t)MUL0 * (uint64_t)c0;
        uint64_t p1 = (uint64_t)MUL1 * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

static void seed_key(uint64_t seed, uint32_t key[2])
{
    key[0] = (uint32_t)(seed & 0xFFFFFFFFu);
    key[1] = (uint32_t)(seed >> 32);
}

/* ------------------------------------------------------------------------ */
/* Section 4.3: sigma ~ S_G, one per (task, group).  Fisher-Yates from the   */
/* top, random words taken from consecutive Philox blocks in output order,   */
/* reduced to [0, k] by multiply-shift.                                      */
/* sigma[k] = index (within the group) of the member that lands on slot k.   */
/* ------------------------------------------------------------------------ */
void ro_permutation(uint64_t seed, uint32_t task_id, uint32_t group_index,
                    uint32_t G, uint32_t *sigma)
{
    uint32_t key[2], ctr[4], blk[4];
    uint32_t n_block = 0, used = 4;
    seed_key(seed, key);
    for (uint32_t k = 0; k < G; ++k) sigma[k] = k;
    for (uint32_t k = G; k-- > 1;) {
        if (used == 4) {
            ctr[0] = n_block++; ctr[1] = group_index; ctr[2] = RO_TAG_PERM; ctr[3] = task_id;
            ro_philox4x32_10(ctr, key, blk);
            used = 0;
        }
        uint32_t r = blk[used++];
        uint32_t j = (uint32_t)(((uint64_t)r * (uint64_t)(k + 1)) >> 32);
        uint32_t t = sigma[k]; sigma[k] = sigma[j]; sigma[j] = t;
    }
}

/* ------------------------------------------------------------------------ */
/* Section 4.4: diagonal entry of D for (task, slot, column): +1 or -1 with  */
/* equal probability.  One Philox block holds the bits of 128 columns.       */
/* ------------------------------------------------------------------------ */
int ro_sign(uint64_t seed, uint32_t task_id, uint32_t slot, uint32_t col)
{
    uint32_t key[2], ctr[4], blk[4];
    seed_key(seed, key);
    ctr[0] = col >> 7; ctr[1] = slot; ctr[2] = RO_TAG_SIGN; ctr[3] = task_id;
    ro_philox4x32_10(ctr, key, blk);
    uint32_t bit = (blk[(col >> 5) & 3u] >> (col & 31u)) & 1u;
    return bit ? -1 : +1;
}

void ro_sign_row(uint64_t seed, uint32_t task_id, uint32_t slot, uint32_t cols, int8_t *out)
{
    for (uint32_t c = 0; c < cols; ++c) out[c] = (int8_t)ro_sign(seed, task_id, slot, c);
}

/* ------------------------------------------------------------------------ */
/* Section 5.5, the "RD" context matrix: a diagonal with (approximately)     */
/* standard normal entries instead of +-1; not orthogonal, and its inverse   */
/* divides.  The paper names no generator.  Here: the sum of twelve uniforms */
/* minus six (mean 0, variance 1), every step an exactly rounded fp32        */
/* operation so that any IEEE machine gets the same bits: the twelve words   */
/* of Philox blocks 3c, 3c+1, 3c+2 of the (slot, task) stream, each reduced  */
/* to u = (word >> 8) * 2^-24, added left to right.  A zero (which could not */
/* be inverted) is replaced by one.                                          */
/* ------------------------------------------------------------------------ */
float ro_gauss(uint64_t seed, uint32_t task_id, uint32_t slot, uint32_t col)
{
    uint32_t key[2], ctr[4], blk[4];
    float sum = 0.0f;
    seed_key(seed, key);
    for (uint32_t b = 0; b < 3; ++b) {
        ctr[0] = 3u * col + b; ctr[1] = slot; ctr[2] = RO_TAG_GAUS; ctr[3] = task_id;
        ro_philox4x32_10(ctr, key, blk);
        for (int w = 0; w < 4; ++w) {
            float u = (float)(blk[w] >> 8) * (1.0f / 16777216.0f); /* exact: 24 bits times a power of two */
            sum = sum + u;                                          /* one rounding */
        }
    }
    float g = sum - 6.0f;
    return g == 0.0f ? 1.0f : g;
}

/* ------------------------------------------------------------------------ */
/* Per-task layer tables over the whole model.                               */
/*   src_of_slot[l] = layer whose delta lands on slot l   (sigma)            */
/*   slot_of_pos[p] = slot that holds layer p's delta     (sigma^-1)         */
/* Group members are the layers carrying that group id, in layer order.      */
/* Returns 0, or -1 if a group id is out of range / allocation fails.        */
/* ------------------------------------------------------------------------ */
/* 1 if the layer's position inside its group is one the skip rate selects. */
static int takes_part(uint32_t n_layers, const uint32_t *group, const uint32_t *gflags, uint32_t l)
{
    uint32_t j = 0, k = RO_SKIP(gflags[group[l]]);
    for (uint32_t a = 0; a < l && a < n_layers; ++a)
        if (group[a] == group[l]) ++j;
    return k <= 1 || j % k == 0;
}

/* 1 if slot l is sign-flipped (Section 4.4, restricted by the skip rate). */
int ro_layer_flips(uint32_t n_layers, const uint32_t *group, const uint32_t *gflags, uint32_t l)
{
    return (gflags[group[l]] & RO_FLIP) != 0 && takes_part(n_layers, group, gflags, l);
}

/* 1 if slot l carries the Gaussian-like context instead (restricted by the skip rate likewise). */
int ro_layer_gauss(uint32_t n_layers, const uint32_t *group, const uint32_t *gflags, uint32_t l)
{
    return (gflags[group[l]] & RO_GAUSS) != 0 && takes_part(n_layers, group, gflags, l);
}

int ro_task_tables(uint32_t n_layers, const uint32_t *group, uint32_t n_groups,
                   const uint32_t *gflags, uint64_t seed, uint32_t task_id,
                   uint32_t *src_of_slot, uint32_t *slot_of_pos)
{
    uint32_t *members = (uint32_t *)malloc(sizeof(uint32_t) * (n_layers + 1));
    uint32_t *sigma = (uint32_t *)malloc(sizeof(uint32_t) * (n_layers + 1));
    if (!members || !sigma) { free(members); free(sigma); return -1; }
    for (uint32_t l = 0; l < n_layers; ++l) {
        if (group[l] >= n_groups) { free(members); free(sigma); return -1; }
        src_of_slot[l] = l;
        slot_of_pos[l] = l;
    }
    for (uint32_t g = 0; g < n_groups; ++g) {
        /* the participating members of the group, in layer order */
        uint32_t n = 0;
        for (uint32_t l = 0; l < n_layers; ++l)
            if (group[l] == g && takes_part(n_layers, group, gflags, l)) members[n++] = l;
        if (n < 2) continue;
        if (gflags[g] & RO_SHUFFLE) {
            ro_permutation(seed, task_id, g, n, sigma);
        } else if (gflags[g] & RO_SHIFT) {
            uint32_t shift = 1u + task_id % (n - 1u);
            for (uint32_t k = 0; k < n; ++k) sigma[k] = (k + n - shift) % n;
        } else {
            continue;
        }
        for (uint32_t k = 0; k < n; ++k) {
            src_of_slot[members[k]] = members[sigma[k]];
            slot_of_pos[members[sigma[k]]] = members[k];
        }
    }
    free(members);
    free(sigma);
    return 0;
}

/* ------------------------------------------------------------------------ */
/* bf16 <-> fp32                                                             */
/* ------------------------------------------------------------------------ */
static float bf16_to_f32(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

uint16_t ro_f32_to_bf16(float f)
{
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu) != 0u)
        return (uint16_t)((u >> 16) | 0x0040u); /* NaN stays NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb; /* round to nearest, ties to even; carries into Inf */
    return (uint16_t)(u >> 16);
}

static float load_elem(const void *p, int dtype, size_t i)
{
    if (dtype == RO_BF16) return bf16_to_f32(((const uint16_t *)p)[i]);
    return ((const float *)p)[i];
}

/* ------------------------------------------------------------------------ */
/* x = T_i(d_i) restricted to one slot l: the shuffled, sign-flipped delta.  */
/* x[r,c] = s_i(l,c) * ( W_i[src][r,c] - W_0[src][r,c] ),  src = sigma_i(l). */
/* base == NULL: `task` already holds the delta (PEFT / LoRA, Section 5.8).  */
/* ------------------------------------------------------------------------ */
static float transformed_delta(const void *w_task, const void *w_base, int dtype,
                               size_t idx, int sign)
{
    float d;
    if (w_base) {
        d = load_elem(w_task, dtype, idx) - load_elem(w_base, dtype, idx); /* one rounding */
    } else {
        d = load_elem(w_task, dtype, idx);
    }
    return sign < 0 ? -d : d;
}

typedef struct {
    uint32_t n_layers;
    const uint32_t *rows, *cols, *group;
    uint32_t n_groups;
    const uint32_t *gflags;
} ro_spec_t;

static int spec_check(const ro_spec_t *s)
{
    for (uint32_t g = 0; g < s->n_groups; ++g)
        if (((s->gflags[g] & RO_SHUFFLE) && (s->gflags[g] & RO_SHIFT)) ||
            ((s->gflags[g] & RO_FLIP) && (s->gflags[g] & RO_GAUSS))) return -3;
    /* all members of a group must have one shape (Section 4.3: same type) */
    for (uint32_t a = 0; a < s->n_layers; ++a) {
        if (s->group[a] >= s->n_groups) return -1;
        for (uint32_t b = a + 1; b < s->n_layers; ++b)
            if (s->group[a] == s->group[b] &&
                (s->rows[a] != s->rows[b] || s->cols[a] != s->cols[b]))
                return -2;
    }
    return 0;
}

/*
 * M[l] (+)= sign_op * T_i(d_i)[l] for one task.  Used by compress (looping
 * over tasks in the given order, starting from +0), add (sign_op=+1) and
 * remove (sign_op=-1).  slot_mask (may be NULL) limits the work to chosen
 * slots so that large cases can be spot-checked.
 */
static float load_m(const void *m, int m_dtype, size_t i) { return load_elem(m, m_dtype, i); }

static void store_m(void *m, int m_dtype, size_t i, float v)
{
    if (m_dtype == RO_BF16) ((uint16_t *)m)[i] = ro_f32_to_bf16(v);
    else ((float *)m)[i] = v;
}

static int accumulate_one(const ro_spec_t *s, int dtype, int m_dtype, int sign_op,
                          uint32_t task_id, uint64_t seed,
                          const void *const *base, const void *const *task,
                          void *const *M, const uint8_t *slot_mask)
{
    uint32_t L = s->n_layers;
    uint32_t *src_of_slot = (uint32_t *)malloc(sizeof(uint32_t) * (L + 1));
    uint32_t *slot_of_pos = (uint32_t *)malloc(sizeof(uint32_t) * (L + 1));
    if (!src_of_slot || !slot_of_pos) { free(src_of_slot); free(slot_of_pos); return -1; }
    if (ro_task_tables(L, s->group, s->n_groups, s->gflags, seed, task_id,
                       src_of_slot, slot_of_pos)) {
        free(src_of_slot); free(slot_of_pos); return -1;
    }
    for (uint32_t l = 0; l < L; ++l) {
        if (slot_mask && !slot_mask[l]) continue;
        uint32_t rows = s->rows[l], cols = s->cols[l];
        uint32_t src = src_of_slot[l];
        int flip = ro_layer_flips(L, s->group, s->gflags, l);
        int gauss = ro_layer_gauss(L, s->group, s->gflags, l);
        int8_t *sg = (int8_t *)malloc(cols ? cols : 1);
        float *gs = (float *)malloc(sizeof(float) * (cols ? cols : 1));
        if (!sg || !gs) { free(sg); free(gs); free(src_of_slot); free(slot_of_pos); return -1; }
        if (flip) ro_sign_row(seed, task_id, l, cols, sg);
        else memset(sg, 1, cols);
        for (uint32_t c = 0; gauss && c < cols; ++c) gs[c] = ro_gauss(seed, task_id, l, c);
        const void *wt = task[src];
        const void *wb = base ? base[src] : NULL;
        void *m = M[l];
#pragma omp parallel for schedule(static)
        for (int64_t r = 0; r < (int64_t)rows; ++r) {
            for (uint32_t c = 0; c < cols; ++c) {
                size_t idx = (size_t)r * cols + c;
                float x = transformed_delta(wt, wb, dtype, idx, sg[c]);
                if (gauss) x = x * gs[c];                    /* Delta D with a Gaussian-like D: one rounding */
                float old = load_m(m, m_dtype, idx);
                float sum = sign_op < 0 ? old - x : old + x; /* one fp32 rounding */
                store_m(m, m_dtype, idx, sum);               /* and one more if M is bf16 */
            }
        }
        free(sg);
        free(gs);
    }
    free(src_of_slot);
    free(slot_of_pos);
    return 0;
}

static ro_spec_t make_spec(uint32_t n_layers, const uint32_t *rows, const uint32_t *cols,
                           const uint32_t *group, uint32_t n_groups, const uint32_t *gflags)
{
    ro_spec_t s;
    s.n_layers = n_layers; s.rows = rows; s.cols = cols; s.group = group;
    s.n_groups = n_groups; s.gflags = gflags;
    return s;
}

/*
 * The sum of several transformed deltas, either from +0.0f (compress) or on top of
 * what M already holds (adding several models at once).
 */
static int sum_models(uint32_t n_layers, const uint32_t *rows, const uint32_t *cols,
                      const uint32_t *group, uint32_t n_groups, const uint32_t *gflags,
                      int dtype, int m_dtype, int from_m, uint32_t n_tasks, const uint32_t *task_ids,
                      const uint64_t *seeds, const void *const *base, const void *const *tasks,
                      void *const *M, const uint8_t *slot_mask)
{
    ro_spec_t s = make_spec(n_layers, rows, cols, group, n_groups, gflags);
    int rc = spec_check(&s);
    if (rc) return rc;
    /* the sum always runs in fp32; a bf16 M receives it rounded once, at the end */
    void **acc = (void **)calloc(n_layers ? n_layers : 1, sizeof(void *));
    if (!acc) return -1;
    for (uint32_t l = 0; l < n_layers; ++l) {
        if (slot_mask && !slot_mask[l]) continue;
        size_t n = (size_t)rows[l] * cols[l];
        if (m_dtype == RO_F32) {
            acc[l] = M[l];
        } else {
            acc[l] = malloc(sizeof(float) * (n ? n : 1));
            if (!acc[l]) { rc = -1; goto done; }
        }
        for (size_t e = 0; e < n; ++e)
            ((float *)acc[l])[e] = from_m ? load_m(M[l], m_dtype, e) : 0.0f;
    }
    for (uint32_t i = 0; i < n_tasks && !rc; ++i)
        rc = accumulate_one(&s, dtype, RO_F32, +1, task_ids[i], seeds[i], base,
                            tasks + (size_t)i * n_layers, acc, slot_mask);
    if (!rc && m_dtype != RO_F32)
        for (uint32_t l = 0; l < n_layers; ++l) {
            if (slot_mask && !slot_mask[l]) continue;
            size_t n = (size_t)rows[l] * cols[l];
            for (size_t e = 0; e < n; ++e) store_m(M[l], m_dtype, e, ((float *)acc[l])[e]);
        }
done:
    if (m_dtype != RO_F32)
        for (uint32_t l = 0; l < n_layers; ++l) free(acc[l]);
    free(acc);
    return rc;
}

/*
 * compress (Section 4, first display; Section 4.4 first display):
 *   M = sum_{i in given order} T_i(W_i - W_0), every slot started from +0.0f.
 * tasks is a flattened [n_tasks][n_layers] array of host pointers.
 */
int ro_compress(uint32_t n_layers, const uint32_t *rows, const uint32_t *cols,
                const uint32_t *group, uint32_t n_groups, const uint32_t *gflags,
                int dtype, int m_dtype, uint32_t n_tasks, const uint32_t *task_ids, const uint64_t *seeds,
                const void *const *base, const void *const *tasks,
                void *const *M, const uint8_t *slot_mask)
{
    return sum_models(n_layers, rows, cols, group, n_groups, gflags, dtype, m_dtype, 0, n_tasks, task_ids, seeds,
                      base, tasks, M, slot_mask);
}

/*
 * Several models added in one step (Section 5.7, the hot swap applied to a set):
 *   M <- M + T_a(d_a) + T_b(d_b) + ...   summed in fp32 in the given order, starting from M.
 * With an fp32 M this is what the same ro_add_model calls give one after the other; a bf16 M
 * is widened once, summed in fp32 and rounded once at the end.
 */
int ro_add_models(uint32_t n_layers, const uint32_t *rows, const uint32_t *cols,
                  const uint32_t *group, uint32_t n_groups, const uint32_t *gflags,
                  int dtype, int m_dtype, uint32_t n_tasks, const uint32_t *task_ids, const uint64_t *seeds,
                  const void *const *base, const void *const *tasks,
                  void *const *M, const uint8_t *slot_mask)
{
    return sum_models(n_layers, rows, cols, group, n_groups, gflags, dtype, m_dtype, 1, n_tasks, task_ids, seeds,
                      base, tasks, M, slot_mask);
}

/* Model hot swapping (Section 5.7): M <- M + T_j(d_j)  /  M <- M - T_j(d_j). */
int ro_add_model(uint32_t n_layers, const uint32_t *rows, const uint32_t *cols,
                 const uint32_t *group, uint32_t n_groups, const uint32_t *gflags,
                 int dtype, int m_dtype, uint32_t task_id, uint64_t seed,
                 const void *const *base, const void *const *task,
                 void *const *M, const uint8_t *slot_mask)
{
    ro_spec_t s = make_spec(n_layers, rows, cols, group, n_groups, gflags);
    int rc = spec_check(&s);
    if (rc) return rc;
    return accumulate_one(&s, dtype, m_dtype, +1, task_id, seed, base, task, M, slot_mask);
}

int ro_remove_model(uint32_t n_layers, const uint32_t *rows, const uint32_t *cols,
                    const uint32_t *group, uint32_t n_groups, const uint32_t *gflags,
                    int dtype, int m_dtype, uint32_t task_id, uint64_t seed,
                    const void *const *base, const void *const *task,
                    void *const *M, const uint8_t *slot_mask)
{
    ro_spec_t s = make_spec(n_layers, rows, cols, group, n_groups, gflags);
    int rc = spec_check(&s);
    if (rc) return rc;
    return accumulate_one(&s, dtype, m_dtype, -1, task_id, seed, base, task, M, slot_mask);
}

/*
 * retrieve (Section 4, second display; Section 4.4 second display):
 *   What_t = W_0 + lambda * T_t^-1(M).
 * T_t^-1 = P_t^-1 o D_t: undo the flip in M's frame (D is its own inverse),
 * then send slot l back to the layer it came from.  For layer position p:
 *   l = sigma_t^-1(p);  out[p][r,c] = fma(lambda, s_t(l,c) * M[l][r,c], W_0[p][r,c]).
 * out is fp32 or bf16 (round to nearest even).  pos_mask (may be NULL) limits
 * the work to chosen layer positions.
 */
int ro_retrieve(uint32_t n_layers, const uint32_t *rows, const uint32_t *cols,
                const uint32_t *group, uint32_t n_groups, const uint32_t *gflags,
                int dtype, int m_dtype, int out_dtype, uint32_t task_id, uint64_t seed, float lambda,
                const void *const *base, const void *const *M,
                void *const *out, const uint8_t *pos_mask)
{
    ro_spec_t s = make_spec(n_layers, rows, cols, group, n_groups, gflags);
    int rc = spec_check(&s);
    if (rc) return rc;
    uint32_t L = n_layers;
    uint32_t *src_of_slot = (uint32_t *)malloc(sizeof(uint32_t) * (L + 1));
    uint32_t *slot_of_pos = (uint32_t *)malloc(sizeof(uint32_t) * (L + 1));
    if (!src_of_slot || !slot_of_pos) { free(src_of_slot); free(slot_of_pos); return -1; }
    if (ro_task_tables(L, group, n_groups, gflags, seed, task_id, src_of_slot, slot_of_pos)) {
        free(src_of_slot); free(slot_of_pos); return -1;
    }
    for (uint32_t p = 0; p < L; ++p) {
        if (pos_mask && !pos_mask[p]) continue;
        uint32_t nr = rows[p], nc = cols[p];
        uint32_t l = slot_of_pos[p];
        int flip = ro_layer_flips(L, group, gflags, l);
        int gauss = ro_layer_gauss(L, group, gflags, l);
        int8_t *sg = (int8_t *)malloc(nc ? nc : 1);
        float *gs = (float *)malloc(sizeof(float) * (nc ? nc : 1));
        if (!sg || !gs) { free(sg); free(gs); free(src_of_slot); free(slot_of_pos); return -1; }
        if (flip) ro_sign_row(seed, task_id, l, nc, sg);
        else memset(sg, 1, nc);
        for (uint32_t c = 0; gauss && c < nc; ++c) gs[c] = ro_gauss(seed, task_id, l, c);
        const void *m = M[l];
        const void *wb = base[p];
        void *o = out[p];
#pragma omp parallel for schedule(static)
        for (int64_t r = 0; r < (int64_t)nr; ++r) {
            for (uint32_t c = 0; c < nc; ++c) {
                size_t idx = (size_t)r * nc + c;
                float mv = load_m(m, m_dtype, idx);
                float signed_m = sg[c] < 0 ? -mv : mv;
                if (gauss) signed_m = mv / gs[c];            /* D^-1 of a diagonal D divides: one rounding */
                float y = fmaf(lambda, signed_m, load_elem(wb, dtype, idx));
                if (out_dtype == RO_BF16) ((uint16_t *)o)[idx] = ro_f32_to_bf16(y);
                else ((float *)o)[idx] = y;
            }
        }
        free(sg);
        free(gs);
    }
    free(src_of_slot);
    free(slot_of_pos);
    return 0;
}

/*
 * A linear layer applied with a retrieved weight that is never formed
 * (Section 4, second display, inserted into y = x What^T; Section 1 motivates
 * serving many models from one store):
 *   y[b][r] = sum_c x[b][c] * ( W_0[p][r,c] + lambda * s_t(l,c) * M[l][r,c] ),   l = sigma_t^-1(p).
 * Everything is widened to double and summed in double, columns ascending: this
 * is the definition, not a model of any particular arithmetic.  x is
 * [n_tokens, cols] in the storage type; y and y_abs are [n_tokens, rows]
 * doubles; y_abs (may be NULL) receives sum_c |x| * (|W_0| + |lambda * M|), the
 * scale against which a finite-precision result is judged.
 */
int ro_linear(uint32_t n_layers, const uint32_t *rows, const uint32_t *cols,
              const uint32_t *group, uint32_t n_groups, const uint32_t *gflags,
              int dtype, int m_dtype, uint32_t task_id, uint64_t seed, float lambda, uint32_t p,
              const void *x, uint32_t n_tokens, const void *const *base, const void *const *M,
              double *y, double *y_abs)
{
    ro_spec_t s = make_spec(n_layers, rows, cols, group, n_groups, gflags);
    int rc = spec_check(&s);
    if (rc) return rc;
    uint32_t L = n_layers;
    if (p >= L) return -1;
    for (uint32_t g = 0; g < n_groups; ++g)
        if (gflags[g] & RO_GAUSS) return -4;   /* defined for the orthogonal contexts only */
    uint32_t *src_of_slot = (uint32_t *)malloc(sizeof(uint32_t) * (L + 1));
    uint32_t *slot_of_pos = (uint32_t *)malloc(sizeof(uint32_t) * (L + 1));
    if (!src_of_slot || !slot_of_pos) { free(src_of_slot); free(slot_of_pos); return -1; }
    if (ro_task_tables(L, group, n_groups, gflags, seed, task_id, src_of_slot, slot_of_pos)) {
        free(src_of_slot); free(slot_of_pos); return -1;
    }
    uint32_t nr = rows[p], nc = cols[p];
    uint32_t l = slot_of_pos[p];
    int8_t *sg = (int8_t *)malloc(nc ? nc : 1);
    if (!sg) { free(src_of_slot); free(slot_of_pos); return -1; }
    if (ro_layer_flips(L, group, gflags, l)) ro_sign_row(seed, task_id, l, nc, sg);
    else memset(sg, 1, nc);
    const void *m = M[l];
    const void *wb = base[p];
    const double lam = (double)lambda;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < (int64_t)n_tokens; ++b) {
        for (uint32_t r = 0; r < nr; ++r) {
            double acc = 0.0, mag = 0.0;
            for (uint32_t c = 0; c < nc; ++c) {
                size_t idx = (size_t)r * nc + c;
                double xv = (double)load_elem(x, dtype, (size_t)b * nc + c);
                double w0 = (double)load_elem(wb, dtype, idx);
                double mv = (double)load_m(m, m_dtype, idx);
                acc += xv * (w0 + lam * (sg[c] < 0 ? -mv : mv));
                mag += fabs(xv) * (fabs(w0) + fabs(lam * mv));
            }
            y[(size_t)b * nr + r] = acc;
            if (y_abs) y_abs[(size_t)b * nr + r] = mag;
        }
    }
    free(sg);
    free(src_of_slot);
    free(slot_of_pos);
    return 0;
}

/*
 * Gram matrix of the transformed deltas (Section 3: the interference norm is a
 * function of the inner products of the deltas; Section 4: every O_i is
 * orthogonal, so the deltas that interfere at retrieval have the inner products
 * of the transformed deltas):
 *   gram[i*n + j] = sum over slots l and elements (r,c) of x_i * x_j,
 *   x_i = s_i(l,c) * (W_i[sigma_i(l)][r,c] - W_0[sigma_i(l)][r,c])   (the fp32 value compress sums)
 * accumulated in double, element by element.
 */
int ro_delta_gram(uint32_t n_layers, const uint32_t *rows, const uint32_t *cols,
                  const uint32_t *group, uint32_t n_groups, const uint32_t *gflags,
                  int dtype, uint32_t n_tasks, const uint32_t *task_ids, const uint64_t *seeds,
                  const void *const *base, const void *const *tasks, double *gram)
{
    for (uint32_t g = 0; g < n_groups; ++g)
        if (gflags[g] & RO_GAUSS) return -4;   /* the interference identity rests on orthogonal transforms */
    ro_spec_t s = make_spec(n_layers, rows, cols, group, n_groups, gflags);
    int rc = spec_check(&s);
    if (rc) return rc;
    uint32_t L = n_layers, n = n_tasks;
    uint32_t *src = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)(L + 1) * (n + 1));
    uint32_t *pos = (uint32_t *)malloc(sizeof(uint32_t) * (L + 1));
    float *x = (float *)malloc(sizeof(float) * (n + 1));
    if (!src || !pos || !x) { free(src); free(pos); free(x); return -1; }
    for (uint32_t i = 0; i < n; ++i)
        if (ro_task_tables(L, group, n_groups, gflags, seeds[i], task_ids[i], src + (size_t)i * L, pos)) {
            free(src); free(pos); free(x); return -1;
        }
    for (size_t e = 0; e < (size_t)n * n; ++e) gram[e] = 0.0;
    for (uint32_t l = 0; l < L; ++l) {
        uint32_t nr = rows[l], nc = cols[l];
        int flip = ro_layer_flips(L, group, gflags, l);
        int8_t *sg = (int8_t *)malloc((size_t)(nc ? nc : 1) * (n ? n : 1));
        if (!sg) { free(src); free(pos); free(x); return -1; }
        for (uint32_t i = 0; i < n; ++i) {
            if (flip) ro_sign_row(seeds[i], task_ids[i], l, nc, sg + (size_t)i * nc);
            else memset(sg + (size_t)i * nc, 1, nc);
        }
        for (uint32_t r = 0; r < nr; ++r)
            for (uint32_t c = 0; c < nc; ++c) {
                size_t idx = (size_t)r * nc + c;
                for (uint32_t i = 0; i < n; ++i) {
                    uint32_t sl = src[(size_t)i * L + l];
                    x[i] = transformed_delta(tasks[(size_t)i * L + sl], base ? base[sl] : NULL, dtype, idx, sg[(size_t)i * nc + c]);
                }
                for (uint32_t i = 0; i < n; ++i)
                    for (uint32_t j = 0; j < n; ++j) gram[(size_t)i * n + j] += (double)x[i] * (double)x[j];
            }
        free(sg);
    }
    free(src); free(pos); free(x);
    return 0;
}

int ro_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void ro_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
