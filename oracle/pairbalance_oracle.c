/*
 * CPU oracle for the CD-GraB PairBalance ordering computation.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain fp64 statement of what the
 * CUDA library must compute.  It shares no code with the CUDA path and must never be
 * called from it; only the tests, the smoke check and the benchmark's CPU-baseline
 * leg may build or call it.
 *
 * What it follows (arXiv 2302.00845; algorithms numbered in order of appearance):
 *   - loops and front/back pointers: Algorithm 7, "Server-side PairBalance over a set
 *     of vectors (one step)" (Appendix B.1): outer loop over example positions j,
 *     inner loop over workers i = 1..m, a pair consumed at every even j;
 *   - the sign rule: Algorithm 6, "Balancing without normalization" (Appendix A.2):
 *     s = +1 if ||r + c|| < ||r - c|| else -1, then r <- r + s c;
 *   - the pair difference c = z_1 - z_2 with z_1 the earlier vector of the pair:
 *     Algorithm 2, "PairBalance" (Section 3);
 *   - the reorder: Algorithm 1, "Reordering Vectors based on Balanced Signs"
 *     (Section 2): positives to the front in arrival order, negatives to the back in
 *     reverse order;
 *   - epoch reset of the running sum: Algorithm 4, "CD-GraB Parameter Server"
 *     (Section 3.1).
 *
 * Readings taken where the text is silent or garbled:
 *   - the norm is the Euclidean one, so the comparison equals "<r,c> < 0"; the
 *     decision is taken on t = <r,c> in fp64; ties (t == 0, hence r == 0 or c == 0)
 *     give -1 because the printed comparison is strict;
 *   - the back pointer starts at the last position (the printed "1" cannot be meant:
 *     it is decremented), so the back member of pair k lands at position n-1-k;
 *   - the new permutation stores item identifiers pi(j), as the reorder algorithm
 *     appends pi(j);
 *   - each worker's reorder sees only that worker's own signs.
 *
 * A second rule is offered beside the greedy one: RandomizedBalance (Algorithm 2's subroutine,
 * with the bound w of Algorithm 5), p = 1/2 - <r,c>/(2w), s = +1 with probability p.  The
 * uniform draw is an input, so the oracle stays deterministic.  Algorithm 5's second stopping
 * condition (||r||_inf > w) is not evaluated.
 *
 * Replay mode (tolerance rule of the parity tests): when the caller hands in a sign
 * for a position and |t| <= tau * ||r|| * ||c||, the position is a near-tie, the
 * handed-in sign is adopted and counted; outside that band the oracle keeps its own
 * sign and counts a mismatch if the handed-in sign differs.
 *
 * Sums over d are taken in fixed chunks of CDO_CHUNK elements, each chunk summed left
 * to right, the chunk partials then added left to right, so the result does not
 * depend on the number of OpenMP threads.
 *
 * Parity pins live in tests/test_oracle_pins.py.  Odd n is rejected ("parity
 * unpinned": the paper assumes n even and says nothing about an unpaired item).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define CDO_CHUNK 4096
#define CDO_F32 0
#define CDO_BF16 1

typedef struct {
  int m, n;
  long long d;
  int k;           /* pairs consumed so far in this epoch (per worker) */
  int i_next;      /* next worker expected inside the current pair index */
  int epoch_open;
  double *r;       /* running sum, fp64 [d] */
  double *c;       /* scratch difference [d] */
  double *part;    /* chunk partials, 3 per chunk */
  long long nchunk;
  int32_t *perm_cur;  /* [m][n] */
  int32_t *perm_next; /* [m][n] */
  int8_t *signs;      /* [m][n/2] adopted signs */
  int8_t *own;        /* [m][n/2] the oracle's own (no-replay) decision at that state */
  double *t;          /* [m][n/2] <r,c> before the update */
  double *rn;         /* [m][n/2] ||r|| before the update */
  double *cn;         /* [m][n/2] ||c|| */
  long long near_ties, mismatches;
  long long out_of_bound; /* randomized rule: positions with |<r,c>| > w */
} cdo_t;

static double widen(const void *p, long long x, int dtype) {
  if (dtype == CDO_F32) return (double)((const float *)p)[x];
  /* bfloat16: the upper 16 bits of an IEEE binary32 */
  uint32_t u = ((uint32_t)((const uint16_t *)p)[x]) << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

cdo_t *cdo_create(int m, int n, long long d) {
  if (m < 1 || n < 2 || (n & 1) || d < 1) return NULL;
  cdo_t *s = (cdo_t *)calloc(1, sizeof(cdo_t));
  if (!s) return NULL;
  s->m = m; s->n = n; s->d = d;
  s->nchunk = (d + CDO_CHUNK - 1) / CDO_CHUNK;
  size_t np = (size_t)m * (size_t)(n / 2);
  s->r = (double *)calloc((size_t)d, sizeof(double));
  s->c = (double *)calloc((size_t)d, sizeof(double));
  s->part = (double *)calloc((size_t)s->nchunk * 3, sizeof(double));
  s->perm_cur = (int32_t *)malloc(sizeof(int32_t) * (size_t)m * n);
  s->perm_next = (int32_t *)malloc(sizeof(int32_t) * (size_t)m * n);
  s->signs = (int8_t *)calloc(np, 1);
  s->own = (int8_t *)calloc(np, 1);
  s->t = (double *)calloc(np, sizeof(double));
  s->rn = (double *)calloc(np, sizeof(double));
  s->cn = (double *)calloc(np, sizeof(double));
  if (!s->r || !s->c || !s->part || !s->perm_cur || !s->perm_next || !s->signs ||
      !s->own || !s->t || !s->rn || !s->cn)
    return NULL;
  for (int i = 0; i < m; ++i)
    for (int j = 0; j < n; ++j) s->perm_cur[(size_t)i * n + j] = j;
  return s;
}

void cdo_destroy(cdo_t *s) {
  if (!s) return;
  free(s->r); free(s->c); free(s->part); free(s->perm_cur); free(s->perm_next);
  free(s->signs); free(s->own); free(s->t); free(s->rn); free(s->cn);
  free(s);
}

int cdo_set_perms(cdo_t *s, const int32_t *p) {
  if (!s || !p || s->epoch_open) return -1;
  memcpy(s->perm_cur, p, sizeof(int32_t) * (size_t)s->m * s->n);
  return 0;
}

/* Algorithm 4: the running sum is zeroed and the sign list emptied at every epoch. */
int cdo_begin_epoch(cdo_t *s) {
  if (!s || s->epoch_open) return -1;
  memset(s->r, 0, sizeof(double) * (size_t)s->d);
  s->k = 0; s->i_next = 0; s->epoch_open = 1;
  s->near_ties = 0; s->mismatches = 0; s->out_of_bound = 0;
  return 0;
}

/*
 * One PairBalance call for worker i at the current pair index k: z1 = g_prev (the
 * vector at position 2k of the worker's current order), z2 = g_cur (position 2k+1).
 * Workers must come in the order 0..m-1 inside each pair index (coordinated order).
 * replay = 0: no replay; replay = +1/-1: sign seen elsewhere, adopted inside the tie
 * band given by tau.  Returns the adopted sign, or 0 on misuse.
 */
static int balance_core(cdo_t *s, int i, const void *g_prev, const void *g_cur, int dtype,
                        int replay, double tau, int randomized, double u, double w) {
  if (!s || !s->epoch_open || i != s->i_next || s->k >= s->n / 2) return 0;
  const long long d = s->d;
  const long long nchunk = s->nchunk;
  double *r = s->r, *c = s->c, *part = s->part;

#pragma omp parallel for schedule(static)
  for (long long ch = 0; ch < nchunk; ++ch) {
    long long lo = ch * CDO_CHUNK, hi = lo + CDO_CHUNK;
    if (hi > d) hi = d;
    double t = 0.0, rr = 0.0, cc = 0.0;
    for (long long x = lo; x < hi; ++x) {
      double cx = widen(g_prev, x, dtype) - widen(g_cur, x, dtype); /* c = z1 - z2 */
      c[x] = cx;
      t += r[x] * cx;
      rr += r[x] * r[x];
      cc += cx * cx;
    }
    part[3 * ch + 0] = t; part[3 * ch + 1] = rr; part[3 * ch + 2] = cc;
  }
  double t = 0.0, rr = 0.0, cc = 0.0;
  for (long long ch = 0; ch < nchunk; ++ch) {
    t += part[3 * ch + 0]; rr += part[3 * ch + 1]; cc += part[3 * ch + 2];
  }
  /* ||r+c||^2 - ||r-c||^2 = 4<r,c>:  "+1 if ||r+c|| < ||r-c||, else -1". */
  int own = (t < 0.0) ? +1 : -1;
  int sgn = own;
  double rn = sqrt(rr), cn = sqrt(cc);
  if (randomized) {
    /* Algorithm 2's subroutine with the bound w of Algorithm 5 made explicit:
     * p = 1/2 - <r,c>/(2w); +1 with probability p, drawn as "u < p" from the uniform u handed in.
     * |<r,c>| > w is where Algorithm 5 would stop; here p leaves [0,1], the draw becomes
     * deterministic (and equal to the greedy sign) and the event is counted. */
    const double p = 0.5 - t / (2.0 * w);
    own = (u < p) ? +1 : -1;
    sgn = own;
    if (fabs(t) > w) s->out_of_bound++;
    if (replay == 1 || replay == -1) {
      /* an error dt in <r,c> moves p by dt/(2w): the tie band in terms of u - p */
      if (fabs(u - p) > tau * rn * cn / (2.0 * w)) {
        if (replay != own) s->mismatches++;
      } else {
        s->near_ties++;
        sgn = replay;
      }
    }
  } else if (replay == 1 || replay == -1) {
    if (fabs(t) > tau * rn * cn) {
      if (replay != own) s->mismatches++;
    } else {
      s->near_ties++;
      sgn = replay;
    }
  }
  const double sd = (double)sgn;
#pragma omp parallel for schedule(static)
  for (long long x = 0; x < d; ++x) r[x] += sd * c[x]; /* r <- r + s c */

  const int n = s->n, k = s->k;
  size_t pos = (size_t)i * (size_t)(n / 2) + (size_t)k;
  s->signs[pos] = (int8_t)sgn; s->own[pos] = (int8_t)own;
  s->t[pos] = t; s->rn[pos] = rn; s->cn[pos] = cn;

  /* front pointer = k, back pointer = n-1-k for this worker */
  const int32_t *pc = s->perm_cur + (size_t)i * n;
  int32_t *pn = s->perm_next + (size_t)i * n;
  if (sgn == +1) { pn[k] = pc[2 * k];     pn[n - 1 - k] = pc[2 * k + 1]; }
  else           { pn[k] = pc[2 * k + 1]; pn[n - 1 - k] = pc[2 * k]; }

  s->i_next++;
  if (s->i_next == s->m) { s->i_next = 0; s->k++; }
  return sgn;
}

int cdo_balance_one(cdo_t *s, int i, const void *g_prev, const void *g_cur, int dtype,
                    int replay, double tau) {
  return balance_core(s, i, g_prev, g_cur, dtype, replay, tau, 0, 0.0, 1.0);
}

/* RandomizedBalance for worker i: as cdo_balance_one, with the sign drawn from the uniform u
 * in [0,1) and the bound w > 0. */
int cdo_balance_one_randomized(cdo_t *s, int i, const void *g_prev, const void *g_cur, int dtype,
                               double u, double w, int replay, double tau) {
  if (!(w > 0.0)) return 0;
  return balance_core(s, i, g_prev, g_cur, dtype, replay, tau, 1, u, w);
}

/*
 * The uniform draw of RandomizedBalance ("with probability p", Algorithm 2's subroutine) as a
 * function of (seed, epoch, pair index k, worker i), so that a randomized epoch can be repeated:
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3",
 * SC 2011, section on Philox), written from the published definition.  One round maps the
 * counter (c0,c1,c2,c3) under the key (k0,k1) to
 *   (hi(M1*c2) ^ c1 ^ k0,  lo(M1*c2),  hi(M0*c0) ^ c3 ^ k1,  lo(M0*c0))
 * with M0 = 0xD2511F53, M1 = 0xCD9E8D57; after each round the key advances by the Weyl constants
 * (0x9E3779B9, 0xBB67AE85).  Ten rounds.  Pinned by the known-answer vectors published with the
 * generator (tests/golden/philox4x32_10_kat.txt).
 */
void cdo_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* u in [0,1) for (seed, epoch, k, i): counter (i, k, epoch, 0), key = the two halves of the seed,
 * the top 24 bits of the first output word times 2^-24 (exact in single precision). */
double cdo_uniform(unsigned long long seed, unsigned epoch, unsigned k, unsigned i) {
  const uint32_t ctr[4] = {i, k, epoch, 0u}, key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t out[4];
  cdo_philox4x32_10(ctr, key, out);
  return (double)(out[0] >> 8) * (1.0 / 16777216.0);
}

/*
 * One whole step: grads is [2][m][d] (slab 0 = earlier position of each pair, slab 1
 * = later), replay is NULL or m signs.
 */
int cdo_step(cdo_t *s, const void *grads, int dtype, const int8_t *replay, double tau) {
  if (!s || !grads || !s->epoch_open || s->i_next != 0) return -1;
  size_t es = (dtype == CDO_F32) ? 4 : 2;
  const char *base = (const char *)grads;
  for (int i = 0; i < s->m; ++i) {
    const void *gp = base + ((size_t)i * (size_t)s->d) * es;
    const void *gc = base + (((size_t)s->m + i) * (size_t)s->d) * es;
    if (cdo_balance_one(s, i, gp, gc, dtype, replay ? replay[i] : 0, tau) == 0) return -1;
  }
  return 0;
}

/* End of epoch: the next permutations become the current ones. */
int cdo_end_epoch(cdo_t *s, int32_t *perms_out) {
  if (!s || !s->epoch_open || s->k != s->n / 2 || s->i_next != 0) return -1;
  size_t bytes = sizeof(int32_t) * (size_t)s->m * s->n;
  if (perms_out) memcpy(perms_out, s->perm_next, bytes);
  memcpy(s->perm_cur, s->perm_next, bytes);
  s->epoch_open = 0;
  return 0;
}

void cdo_get_r(const cdo_t *s, double *out) { memcpy(out, s->r, sizeof(double) * (size_t)s->d); }
void cdo_get_signs(const cdo_t *s, int8_t *out) { memcpy(out, s->signs, (size_t)s->m * (s->n / 2)); }
void cdo_get_own_signs(const cdo_t *s, int8_t *out) { memcpy(out, s->own, (size_t)s->m * (s->n / 2)); }
void cdo_get_perm_cur(const cdo_t *s, int32_t *out) { memcpy(out, s->perm_cur, sizeof(int32_t) * (size_t)s->m * s->n); }
void cdo_get_perm_next(const cdo_t *s, int32_t *out) { memcpy(out, s->perm_next, sizeof(int32_t) * (size_t)s->m * s->n); }
void cdo_get_trace(const cdo_t *s, double *t, double *rn, double *cn) {
  size_t np = (size_t)s->m * (s->n / 2);
  memcpy(t, s->t, np * sizeof(double));
  memcpy(rn, s->rn, np * sizeof(double));
  memcpy(cn, s->cn, np * sizeof(double));
}
long long cdo_near_ties(const cdo_t *s) { return s->near_ties; }
long long cdo_mismatches(const cdo_t *s) { return s->mismatches; }
long long cdo_out_of_bound(const cdo_t *s) { return s->out_of_bound; }
int cdo_pairs_done(const cdo_t *s) { return s->k; }
int cdo_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
