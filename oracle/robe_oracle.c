/*
 * ROBE-Z oracle: a plain, slow, CPU-only evaluation of the ROBE-Z embedding
 * lookup and its gradient, written from the paper's definitions
 * (arXiv 2108.02191, Section 3.1 "ROBE-D", Section 3.2 "ROBE-Z", the idx / h / g
 * equations in those sections, and the backward equation of Section 3.1).
 *
 * THIS IS TEST INFRASTRUCTURE.  Nothing in the product library calls it, and it
 * shares no code, header, table or constant generator with the CUDA path.  It is
 * used by the test-suite, by the smoke check and by the benchmark's CPU-baseline
 * leg only.
 *
 * Every integer quantity is evaluated with the C `%` operator on
 * `unsigned __int128`; there is no Mersenne folding, no reciprocal trick and no
 * blocking beyond the chunk structure the paper itself states.
 *
 * Readings of the paper taken here (each is listed again in the design notes):
 *   - idx(e,x,i) = (h(e,x,floor(i/Z)) + (i mod Z)) mod m: the in-chunk offset is
 *     added outside the hash (the ROBE-D form of Section 3.1, the slice form of
 *     Section 3.2 and the Figure 2 caption force this; the printed idx equation
 *     of Section 3.2 has a misplaced parenthesis).
 *   - "(..) mod P mod |M|" is ((..) mod P) mod |M|.
 *   - e, x, c and i are 0-based.
 *   - P = 2^61 - 1 (Section 3.2 asks for a large prime and names none); the
 *     multipliers are in [1, P-1], the additive terms in [0, P-1] (Section 3.2).
 *   - the sign hash g is optional and off by default (Section 4.1 and the
 *     appendix both say it is not used in practice).
 *   - pooling over a bag is a sequential fp32 sum in bag order (the paper's data
 *     are one-hot, so this part is a definition of this library, not the paper's).
 *   - Z > d (Section 3.2, last paragraph: a chunk may span several embeddings;
 *     the appendix cuts the row-wise flattened table into chunks of Z) is taken
 *     for d dividing Z: R = Z/d consecutive rows of a table share one
 *     block, row x is the piece [(x mod R) d, (x mod R) d + d) of the block that
 *     starts at h(e, floor(x/R), 0).
 *
 * Parity pins: the hash arithmetic, the idx mapping, the circular wrap, the
 * Z = d and Z = 1 special cases, the sign range, the adjoint identity that ties
 * backward to forward, gradient-mass conservation and the canonical fp32 order
 * are all pinned by tests that do not call this file's formulas back.
 * Parity unpinned (no value in the paper fixes them; they are this library's own
 * definitions): the numeric values of the hash constants drawn from a seed, the
 * choice P = 2^61 - 1, the bag layout, and the canonical summation order of the
 * deterministic backward.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef unsigned __int128 u128;

#define ORACLE_F32 0
#define ORACLE_BF16 1

/* Index layout of the nine constants every function takes. */
enum { K_P = 0, K_AH, K_BH, K_CH, K_DH, K_AG, K_BG, K_CG, K_DG };

/* ---- constants (Section 3.2: P prime and large, A,B,C in 1..P-1, D in 0..P-1) ---- */

static uint64_t mix_next(uint64_t *state) {
    /* SplitMix64 step (published generator by Steele, Lea, Flood). */
    *state += 0x9E3779B97F4A7C15ULL;
    uint64_t z = *state;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

void robe_oracle_hash_constants(uint64_t seed, uint64_t out[9]) {
    const uint64_t P = (1ULL << 61) - 1ULL;
    uint64_t state = seed;
    out[K_P] = P;
    /* draw order: A_h B_h C_h D_h A_g B_g C_g D_g; a 61-bit draw is rejected and
       redrawn when it falls outside the allowed range */
    for (int k = 1; k <= 8; ++k) {
        int additive = (k == K_DH || k == K_DG);
        for (;;) {
            uint64_t v = mix_next(&state) >> 3;
            if (v >= P) continue;
            if (!additive && v == 0) continue;
            out[k] = v;
            break;
        }
    }
}

int robe_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ---- location mapping (Section 3.2, h and idx equations) ---- */

uint64_t robe_oracle_h(const uint64_t k[9], uint64_t m, uint64_t e, uint64_t x, uint64_t c) {
    u128 t = (u128)k[K_AH] * e + (u128)k[K_BH] * x + (u128)k[K_CH] * c + (u128)k[K_DH];
    uint64_t r = (uint64_t)(t % (u128)k[K_P]);
    return r % m;
}

uint64_t robe_oracle_idx(const uint64_t k[9], uint64_t m, uint64_t Z, uint64_t d, uint64_t e,
                         uint64_t x, uint64_t i) {
    if (Z > d) { /* rows clubbed into one chunk of Z: position x d + i of the flattened table */
        uint64_t R = Z / d;
        return (robe_oracle_h(k, m, e, x / R, 0) + (x % R) * d + i) % m;
    }
    uint64_t c = i / Z; /* chunk id    */
    uint64_t o = i % Z; /* offset in it */
    return (robe_oracle_h(k, m, e, x, c) + o) % m;
}

/* The blocks of one embedding, for any Z.  Z <= d: ceil(d/Z) blocks, block c holds elements
   [cZ, min(cZ+Z, d)) and starts at h(e,x,c).  Z > d (d divides Z): ONE block holding all d
   elements; it is the piece of the shared Z-block of rows floor(x/R)R .. +R-1 (R = Z/d) that
   belongs to row x, so it starts (x mod R) d slots after h(e, floor(x/R), 0). */
static uint64_t blocks_per_id(uint64_t Z, uint64_t d) { return Z > d ? 1 : (d + Z - 1) / Z; }

static uint64_t block_len(uint64_t Z, uint64_t d, uint64_t c) {
    if (Z > d) return d;
    return c * Z + Z <= d ? Z : d - c * Z;
}

static uint64_t block_first_elem(uint64_t Z, uint64_t d, uint64_t c) { return Z > d ? 0 : c * Z; }

uint64_t robe_oracle_block_start(const uint64_t k[9], uint64_t m, uint64_t Z, uint64_t d,
                                 uint64_t e, uint64_t x, uint64_t c) {
    if (Z > d) {
        uint64_t R = Z / d;
        return (robe_oracle_h(k, m, e, x / R, 0) + (x % R) * d) % m;
    }
    return robe_oracle_h(k, m, e, x, c);
}

/* sign hash (Section 3.1, g equation): +1 or -1 */
int robe_oracle_g(const uint64_t k[9], uint64_t e, uint64_t x, uint64_t i) {
    u128 t = (u128)k[K_AG] * e + (u128)k[K_BG] * x + (u128)k[K_CG] * i + (u128)k[K_DG];
    uint64_t r = (uint64_t)(t % (u128)k[K_P]);
    return 2 * (int)(r % 2) - 1;
}

static float array_at(const void *array, int dtype, uint64_t j) {
    if (dtype == ORACLE_BF16) {
        /* bf16 is the upper half of an fp32: widening is exact */
        uint32_t bits = (uint32_t)((const uint16_t *)array)[j] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return f;
    }
    return ((const float *)array)[j];
}

/* bag k covers indices[lo..hi) */
static void bag_bounds(const int64_t *offsets, int64_t k, int64_t *lo, int64_t *hi) {
    if (offsets) {
        *lo = offsets[k];
        *hi = offsets[k + 1];
    } else {
        *lo = k;
        *hi = k + 1;
    }
}

/* One output row: E summed over the bag, sequentially, in fp32, the first term
   initialising the accumulator (empty bag -> +0). */
/* Table of bag number `bag`.  Sample-major bags are numbered n*T + e (the default); table-major
 * bags e*B + n, the per-table id lists laid end to end: per_table = B, the number of bags of one
 * table, selects that numbering, per_table = 0 the default. */
static uint64_t table_of(int64_t bag, uint64_t T, int64_t per_table) {
    return per_table ? (uint64_t)(bag / per_table) : (uint64_t)bag % T;
}

static void forward_one_bag(const uint64_t k[9], uint64_t m, uint64_t Z, uint64_t d, uint64_t T,
                            int sign, const void *array, int dtype, const int64_t *indices,
                            const int64_t *offsets, int64_t bag, int64_t per_table, float *row) {
    int64_t lo, hi;
    bag_bounds(offsets, bag, &lo, &hi);
    uint64_t e = table_of(bag, T, per_table);
    for (uint64_t i = 0; i < d; ++i) row[i] = 0.0f;
    for (int64_t p = lo; p < hi; ++p) {
        uint64_t x = (uint64_t)indices[p];
        uint64_t nchunks = blocks_per_id(Z, d);
        for (uint64_t c = 0; c < nchunks; ++c) {
            uint64_t h = robe_oracle_block_start(k, m, Z, d, e, x, c);
            for (uint64_t o = 0; o < block_len(Z, d, c); ++o) {
                uint64_t i = block_first_elem(Z, d, c) + o;
                float v = array_at(array, dtype, (h + o) % m);
                if (sign) v = (float)robe_oracle_g(k, e, x, i) * v;
                row[i] = (p == lo) ? v : row[i] + v;
            }
        }
    }
}

/* Forward over all bags: out[batch*T, d] (Section 3.2 forward; pooling as stated above). */
void robe_oracle_forward(const uint64_t k[9], uint64_t m, uint64_t Z, uint64_t d, uint64_t T,
                         int sign, const void *array, int dtype, const int64_t *indices,
                         const int64_t *offsets, int64_t batch, int64_t per_table, float *out) {
    int64_t nbags = batch * (int64_t)T;
#pragma omp parallel for schedule(static)
    for (int64_t bag = 0; bag < nbags; ++bag)
        forward_one_bag(k, m, Z, d, T, sign, array, dtype, indices, offsets, bag, per_table, out + bag * d);
}

/* Forward for a chosen list of bags only: out[nsel, d]. */
void robe_oracle_forward_bags(const uint64_t k[9], uint64_t m, uint64_t Z, uint64_t d, uint64_t T,
                              int sign, const void *array, int dtype, const int64_t *indices,
                              const int64_t *offsets, const int64_t *bags, int64_t nsel,
                              int64_t per_table, float *out) {
#pragma omp parallel for schedule(static)
    for (int64_t s = 0; s < nsel; ++s)
        forward_one_bag(k, m, Z, d, T, sign, array, dtype, indices, offsets, bags[s], per_table, out + s * d);
}

/* The slots idx(e,x,i) of one embedding, for tests that need the mapping itself. */
void robe_oracle_locate(const uint64_t k[9], uint64_t m, uint64_t Z, uint64_t d, uint64_t e,
                        uint64_t x, uint64_t *slots) {
    for (uint64_t c = 0; c < blocks_per_id(Z, d); ++c) {
        uint64_t h = robe_oracle_block_start(k, m, Z, d, e, x, c);
        for (uint64_t o = 0; o < block_len(Z, d, c); ++o)
            slots[block_first_elem(Z, d, c) + o] = (h + o) % m;
    }
}

/* ---- backward (Section 3.1 backward equation): delta[j] = sum over idx(e,x,i)=j of g * dE ---- */

/* fp64 reference restricted to the slot window [j0, j0+jn): delta64[j-j0] and the
   L1 mass l1[j-j0] = sum |dE| over the same contributions.  Both are ADDED to. */
void robe_oracle_backward_f64(const uint64_t k[9], uint64_t m, uint64_t Z, uint64_t d, uint64_t T,
                              int sign, const float *grad_out, const int64_t *indices,
                              const int64_t *offsets, int64_t batch, int64_t per_table, uint64_t j0,
                              uint64_t jn, double *delta64, double *l1) {
    int64_t nbags = batch * (int64_t)T;
    uint64_t nchunks = blocks_per_id(Z, d);
    for (int64_t bag = 0; bag < nbags; ++bag) {
        int64_t lo, hi;
        bag_bounds(offsets, bag, &lo, &hi);
        uint64_t e = table_of(bag, T, per_table);
        const float *grow = grad_out + bag * (int64_t)d;
        for (int64_t p = lo; p < hi; ++p) {
            uint64_t x = (uint64_t)indices[p];
            for (uint64_t c = 0; c < nchunks; ++c) {
                uint64_t h = robe_oracle_block_start(k, m, Z, d, e, x, c);
                for (uint64_t o = 0; o < block_len(Z, d, c); ++o) {
                    uint64_t i = block_first_elem(Z, d, c) + o;
                    uint64_t j = (h + o) % m;
                    if (j < j0 || j - j0 >= jn) continue;
                    double gsign = sign ? (double)robe_oracle_g(k, e, x, i) : 1.0;
                    delta64[j - j0] += gsign * (double)grow[i];
                    l1[j - j0] += fabs((double)grow[i]);
                }
            }
        }
    }
}

typedef struct {
    uint64_t s; /* block start h(e,x,c)            */
    uint64_t q; /* flat block number p * nchunks + c */
} block_key;

static int block_key_cmp(const void *a, const void *b) {
    const block_key *ka = (const block_key *)a, *kb = (const block_key *)b;
    if (ka->s != kb->s) return ka->s < kb->s ? -1 : 1;
    if (ka->q != kb->q) return ka->q < kb->q ? -1 : 1;
    return 0;
}

/* Canonical fp32 gradient, the order the deterministic GPU variant must reproduce:
   blocks are numbered q = p*nchunks + c in input order, sorted by start s ascending
   (ties keep q ascending), and applied one after another, each slot accumulating
   left to right in fp32 from +0.  Restricted to the window [j0, j0+jn).
   delta[j-j0] is OVERWRITTEN; touched[j-j0] = 1 where at least one term landed.
   Returns 0, or -1 if memory for the key list could not be had. */
int robe_oracle_backward_canonical(const uint64_t k[9], uint64_t m, uint64_t Z, uint64_t d,
                                   uint64_t T, int sign, const float *grad_out,
                                   const int64_t *indices, const int64_t *offsets, int64_t batch,
                                   int64_t per_table, uint64_t j0, uint64_t jn, float *delta,
                                   uint8_t *touched) {
    int64_t nbags = batch * (int64_t)T;
    uint64_t nchunks = blocks_per_id(Z, d);
    int64_t nnz = offsets ? offsets[nbags] : nbags;
    uint64_t nblocks = (uint64_t)nnz * nchunks;
    block_key *keys = (block_key *)malloc((nblocks ? nblocks : 1) * sizeof(block_key));
    int64_t *bag_of = (int64_t *)malloc((nnz ? nnz : 1) * sizeof(int64_t));
    if (!keys || !bag_of) {
        free(keys);
        free(bag_of);
        return -1;
    }
    for (int64_t bag = 0; bag < nbags; ++bag) {
        int64_t lo, hi;
        bag_bounds(offsets, bag, &lo, &hi);
        uint64_t e = table_of(bag, T, per_table);
        for (int64_t p = lo; p < hi; ++p) {
            bag_of[p] = bag;
            for (uint64_t c = 0; c < nchunks; ++c) {
                keys[(uint64_t)p * nchunks + c].s =
                    robe_oracle_block_start(k, m, Z, d, e, (uint64_t)indices[p], c);
                keys[(uint64_t)p * nchunks + c].q = (uint64_t)p * nchunks + c;
            }
        }
    }
    qsort(keys, nblocks, sizeof(block_key), block_key_cmp);
    for (uint64_t j = 0; j < jn; ++j) {
        delta[j] = 0.0f;
        touched[j] = 0;
    }
    for (uint64_t b = 0; b < nblocks; ++b) {
        uint64_t p = keys[b].q / nchunks, c = keys[b].q % nchunks;
        int64_t bag = bag_of[p];
        uint64_t e = table_of(bag, T, per_table);
        uint64_t x = (uint64_t)indices[p];
        const float *grow = grad_out + bag * (int64_t)d;
        for (uint64_t o = 0; o < block_len(Z, d, c); ++o) {
            uint64_t i = block_first_elem(Z, d, c) + o;
            uint64_t j = (keys[b].s + o) % m;
            if (j < j0 || j - j0 >= jn) continue;
            float term = grow[i];
            if (sign) term = (float)robe_oracle_g(k, e, x, i) * term;
            delta[j - j0] = delta[j - j0] + term;
            touched[j - j0] = 1;
        }
    }
    free(keys);
    free(bag_of);
    return 0;
}

/* SGD step (Section 5 trains DLRM with plain SGD): M[j] <- fma(-lr, delta[j], M[j])
   on the slots that received at least one term; other slots keep their bits. */
void robe_oracle_sgd_apply(float *array, const float *delta, const uint8_t *touched, uint64_t n,
                           float lr) {
    for (uint64_t j = 0; j < n; ++j)
        if (touched[j]) array[j] = fmaf(-lr, delta[j], array[j]);
}

/* Dense SGD apply of the data-parallel step (Section 1: the compressed model is trained
   data-parallel, the ranks exchanging one gradient the size of the array; Section 5: SGD):
   M[j] <- fma(-lr, g[j], M[j]) for EVERY slot, g being the gradient summed over the ranks. */
void robe_oracle_dense_sgd_apply(float *array, const float *grad, uint64_t n, float lr) {
    for (uint64_t j = 0; j < n; ++j) array[j] = fmaf(-lr, grad[j], array[j]);
}

/* Dense accumulation used by the deterministic variant: ga[j] <- ga[j] + delta[j]
   on touched slots (one fp32 add). */
void robe_oracle_accumulate(float *grad_array, const float *delta, const uint8_t *touched,
                            uint64_t n) {
    for (uint64_t j = 0; j < n; ++j)
        if (touched[j]) grad_array[j] = grad_array[j] + delta[j];
}

/* Adagrad step (Duchi, Hazan, Singer) on the slots that received at least one term, in fp32, one
   operation at a time, one accumulator per slot:
     s <- s + g^2;  M <- M - lr g / (sqrt(s) + eps)
   Slots without a term keep M and s. */
void robe_oracle_adagrad_apply(float *array, float *sum_sq, const float *delta, const uint8_t *touched,
                               uint64_t n, float lr, float eps) {
    for (uint64_t j = 0; j < n; ++j) {
        if (!touched[j]) continue;
        float g = delta[j];
        float gg = g * g;
        float s = sum_sq[j] + gg;
        sum_sq[j] = s;
        float den = sqrtf(s) + eps;
        float upd = g / den;
        float step = lr * upd;
        array[j] = array[j] - step;
    }
}

/* Adam step (Kingma & Ba, Algorithm 1; Section 5 trains five of the six models with Adam) on
   the slots that received at least one term, in fp32, one operation at a time:
     m1 <- beta1 m1 + (1-beta1) g;  m2 <- beta2 m2 + (1-beta2) g^2
     M  <- M - lr (m1 / bias1) / (sqrt(m2 / bias2) + eps),  bias_k = 1 - beta_k^t (passed in)
   Slots without a term keep M, m1 and m2 (lazy update). */
void robe_oracle_adam_apply(float *array, float *m1, float *m2, const float *delta,
                            const uint8_t *touched, uint64_t n, float lr, float beta1, float beta2,
                            float eps, float bias1, float bias2) {
    for (uint64_t j = 0; j < n; ++j) {
        if (!touched[j]) continue;
        float g = delta[j];
        float a = beta1 * m1[j];
        float b = (1.0f - beta1) * g;
        float m = a + b;
        float c = beta2 * m2[j];
        float gg = g * g;
        float dd = (1.0f - beta2) * gg;
        float v = c + dd;
        m1[j] = m;
        m2[j] = v;
        float mhat = m / bias1;
        float vhat = v / bias2;
        float den = sqrtf(vhat) + eps;
        float upd = mhat / den;
        float step = lr * upd;
        array[j] = array[j] - step;
    }
}
