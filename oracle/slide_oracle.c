/*
 * slide_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded CPU statement of the SLIDE adaptive-sparse
 * training step of a two-layer fully connected network (sparse input ->
 * dense ReLU hidden layer -> LSH-sampled softmax output layer), written
 * from the paper's description (Section 2.1 "The SLIDE Algorithm",
 * Algorithm 1 "D-SLIDE Training", Section 3.5-3.7, Section 4.1).  It is the
 * reference the CUDA library is checked against and shares no code with
 * it.  Only tests, the smoke check and the CPU-baseline leg of the
 * benchmark may call it; the product never does.
 *
 * Every function follows the order of the paper's algorithm and does no
 * blocking, fusion or reordering.  The loops over samples, over neurons and
 * over touched rows carry OpenMP pragmas that only a second build
 * (-fopenmp, used to time the oracle on all host cores) honours; each
 * accumulator still receives the same addends in the same order, so that
 * build is bit-identical to the plain one (pinned in tests).  The scalar type REAL is chosen at
 * compile time: float (the parity target: the paper's networks are fp32
 * and hash codes depend on the exact fp32 hidden activation) or double
 * (used by the gradient and dense-limit pins).
 *
 * Where the paper is silent the reading taken is stated next to the code
 * (marked "reading:").  Pins: tests/test_oracle_*.py (the generator and the initial weights: tests/test_oracle_rng.py).  Unpinned: the
 * paper's accuracy figures (they need its datasets) -- "parity unpinned"
 * for those; no function in this file is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* Which of nthreads workers this one is (0 of 1 in the plain build). */
static void who_am_i(int *tid, int *nthreads) {
#ifdef _OPENMP
  *tid = omp_get_thread_num(); *nthreads = omp_get_num_threads();
#else
  *tid = 0; *nthreads = 1;
#endif
}
int32_t orc_threads(void) {
#ifdef _OPENMP
  return (int32_t)omp_get_max_threads();
#else
  return 1;
#endif
}

#ifndef REAL
#define REAL float
#endif

#define ORC_IS_FLOAT (sizeof(REAL) == sizeof(float))

static REAL r_fma(REAL a, REAL b, REAL c) { return ORC_IS_FLOAT ? (REAL)fmaf((float)a, (float)b, (float)c) : (REAL)fma(a, b, c); }
static REAL r_exp(REAL a) { return ORC_IS_FLOAT ? (REAL)expf((float)a) : (REAL)exp(a); }
static REAL r_log(REAL a) { return ORC_IS_FLOAT ? (REAL)logf((float)a) : (REAL)log(a); }
static REAL r_sqrt(REAL a) { return ORC_IS_FLOAT ? (REAL)sqrtf((float)a) : (REAL)sqrt(a); }

typedef struct {
  int32_t D, H, N;          /* input, hidden, output dimension (Section 4.1: two-layer network) */
  int32_t family;           /* 0 = SimHash / sparse random projections, 1 = DWTA (Section 4.1)   */
  int32_t K, L;             /* K hash functions per table, L tables (Section 4.1)                */
  int32_t bin_size;         /* DWTA bin size, a power of two (reading: 8)                        */
  int32_t srp_nnz;          /* nonzeros per SimHash projection (reading: ceil(H/3))              */
  int32_t bucket_cap;       /* a query sees at most this many ids of a bucket                    */
  int32_t rebuild_period0;  /* first rebuild gap; 0 = never                                      */
  int32_t redraw;           /* draw new hash functions at every rebuild (Algorithm 1, last line) */
  int32_t force_dense;      /* "sparsity is 1" (Section 3.6): every output neuron is active      */
  int32_t max_active;       /* 0 = no limit; otherwise a larger active set is an error           */
  int32_t densify;          /* DWTA: an all-zero bin of a query borrows another bin's position   */
  int32_t budget;           /* Section 3.7: active neurons per sample, labels included; 0 = off   */
  int32_t budget_fill;      /* Section 3.7: an under-full set is topped up with uniform draws     */
  double rebuild_lambda;    /* gap_i = max(1, floor(p0 * exp(lambda * i)))                       */
  double lr, beta1, beta2, eps;   /* Adam (Section 4.1)                                          */
  double init_std;
  uint64_t seed;
  /* LSH-sampled hidden layer (Algorithm 1: active neurons are retrieved for EVERY layer; Section 3.6: a dense layer is
   * the case "sparsity is 1").  hidden_L = 0: the hidden layer is dense.  hidden_L > 0: L tables of hidden_K-bit
   * SimHash codes over the hidden neurons' weight vectors, queried with the sparse input; a query reads at most
   * hidden_cap ids of a bucket. */
  int32_t hidden_K, hidden_L, hidden_cap;
} orc_config;

typedef struct {
  orc_config c;
  int32_t bits;             /* bits of a bucket code */
  int32_t idx_per_fn;       /* srp_nnz (SimHash) or bin_size (DWTA) */
  REAL *W1, *b1, *W2, *b2;
  REAL *mW1, *vW1, *mb1, *vb1, *mW2, *vW2, *mb2, *vb2;
  REAL *dW1, *db1, *dW2, *db2;
  uint8_t *touch1, *touch2;
  int64_t t;                /* Adam step count */
  int64_t r;                /* rebuild count   */
  int64_t next_rebuild;
  int32_t *hash_idx;        /* [K*L][idx_per_fn] */
  int32_t *hash_sign;       /* [K*L][srp_nnz], +1/-1 (SimHash only) */
  int32_t *bucket_off;      /* [L][2^bits + 1] */
  int32_t *bucket_ids;      /* [L][N] */
  /* hidden layer, when it is LSH-sampled */
  int8_t *proj1;            /* [D][hidden_K*hidden_L]: +1 / -1 / 0, the first layer's sparse random projections */
  int32_t *bucket1_off;     /* [hidden_L][2^hidden_K + 1] */
  int32_t *bucket1_ids;     /* [hidden_L][H] */
  uint32_t *codes1;         /* [B][hidden_L] codes of the inputs */
  uint8_t *hact;            /* [B][H] 1 = hidden neuron active for the sample */
  uint8_t *touch1e;         /* [D][H] 1 = weight touched by the batch (input nonzero and hidden neuron active) */
  /* snapshot of the last forward pass (Section 3.6: active neurons, activations, errors) */
  int32_t B;
  REAL *h, *dh;             /* [B][H] */
  uint32_t *codes;          /* [B][L] */
  int64_t *act_ptr;         /* [B+1] */
  int32_t *act_ids;         /* [act_ptr[B]] ascending within a sample */
  REAL *act_z, *act_p, *act_g;
  REAL *loss;               /* [B] */
  int64_t act_capacity;
  int32_t B_capacity;
  /* copies of the last batch (needed by the backward pass) */
  int32_t *row_ptr, *col_idx; REAL *vals; int32_t *label_ptr, *labels;
  int64_t nnz_capacity, lab_capacity;
  int32_t error;            /* 0 ok, 4 active-set overflow, 5 bad index */
} orc;

/* ------------------------------------------------------------------ */
/* Counter-based random numbers: three rounds of the splitmix64 output */
/* function over (seed, stream, r, counter).  The CUDA library carries */
/* its own independent statement of the same definition.               */
/* ------------------------------------------------------------------ */
static uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}
static const uint64_t GOLD = 0x9E3779B97F4A7C15ULL;

/* The output function alone, for the pin against the published splitmix64 outputs:
 * the k-th output of splitmix64 seeded with s is mix64(s + k * GOLD), k = 1, 2, ... */
uint64_t orc_mix64(uint64_t z) { return mix64(z); }

uint64_t orc_rng(uint64_t seed, uint64_t stream, uint64_t r, uint64_t ctr) {
  uint64_t a = mix64(seed + GOLD * (stream + 1));
  uint64_t b = mix64(a + GOLD * (r + 1));
  return mix64(b + GOLD * (ctr + 1));
}
enum { STREAM_W1 = 0, STREAM_W2 = 1, STREAM_HASH = 2, STREAM_PROBE = 3, STREAM_SAMPLE = 4, STREAM_FILL = 5, STREAM_HASH1 = 6 };
enum { DENSIFY_ATTEMPTS = 16 };

static double u01(uint64_t x) { return ((double)(x >> 11) + 0.5) * (1.0 / 9007199254740992.0); }

/* Algorithm 1, line "Initialize layers with randomly generated weights".
 * reading: N(0, init_std^2) by Box-Muller over two counter-based uniforms;
 * biases and Adam moments start at zero. */
static void init_gauss(REAL *w, int64_t n, uint64_t seed, uint64_t stream, double std) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    double u1 = u01(orc_rng(seed, stream, 0, 2 * (uint64_t)i));
    double u2 = u01(orc_rng(seed, stream, 0, 2 * (uint64_t)i + 1));
    w[i] = (REAL)(std * sqrt(-2.0 * log(u1)) * cos(6.283185307179586476925 * u2));
  }
}

static int cmp_i32(const void *a, const void *b) {
  int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
  return (x > y) - (x < y);
}

/* Hash functions for rebuild count r (Algorithm 1: "Rebuild hash tables and
 * hash functions").
 * SimHash (sparse random projections, Section 4.1), reading: projection p
 * has exactly srp_nnz distinct coordinates, chosen by a partial Fisher-Yates
 * shuffle of 0..H-1 and then sorted ascending, each with a sign +1/-1.
 * DWTA (Section 4.1), reading: ceil(K*L*bin/H) random permutations of the
 * H coordinates are concatenated; hash function p reads entries
 * [p*bin, (p+1)*bin) of the concatenation. */
void orc_draw_hash(orc *o, int64_t r) {
  const orc_config *c = &o->c;
  int KL = c->K * c->L, H = c->H;
  int32_t *perm = (int32_t *)malloc(sizeof(int32_t) * (size_t)H);
  if (c->family == 0) {
    int m = c->srp_nnz;
    for (int p = 0; p < KL; ++p) {
      for (int i = 0; i < H; ++i) perm[i] = i;
      for (int i = 0; i < m; ++i) {
        uint64_t u = orc_rng(c->seed, STREAM_HASH, (uint64_t)r, (uint64_t)p * 2u * (uint64_t)m + (uint64_t)i);
        int j = i + (int)(u % (uint64_t)(H - i));
        int32_t tmp = perm[i]; perm[i] = perm[j]; perm[j] = tmp;
      }
      qsort(perm, (size_t)m, sizeof(int32_t), cmp_i32);
      for (int i = 0; i < m; ++i) {
        uint64_t u = orc_rng(c->seed, STREAM_HASH, (uint64_t)r, (uint64_t)p * 2u * (uint64_t)m + (uint64_t)m + (uint64_t)i);
        o->hash_idx[(size_t)p * m + i] = perm[i];
        o->hash_sign[(size_t)p * m + i] = (u & 1u) ? 1 : -1;
      }
    }
  } else {
    int bs = c->bin_size;
    int64_t total = (int64_t)KL * bs;
    int64_t nperm = (total + H - 1) / H;
    for (int64_t q = 0; q < nperm; ++q) {
      for (int i = 0; i < H; ++i) perm[i] = i;
      for (int i = H - 1; i >= 1; --i) {
        uint64_t u = orc_rng(c->seed, STREAM_HASH, (uint64_t)r, (uint64_t)q * (uint64_t)H + (uint64_t)i);
        int j = (int)(u % (uint64_t)(i + 1));
        int32_t tmp = perm[i]; perm[i] = perm[j]; perm[j] = tmp;
      }
      for (int i = 0; i < H; ++i) {
        int64_t e = q * H + i;
        if (e < total) o->hash_idx[e] = perm[i];
      }
    }
  }
  free(perm);
}

/* The L bucket codes of a vector v[H].  The same function hashes queries
 * (v = hidden activation) and neurons (v = weight row; reading: the bias
 * is not hashed).
 * SimHash, reading: s = sum in stored coordinate order, sequential in REAL;
 * bit = (s >= 0); code = sum_k bit_k << k.
 * DWTA, reading: position of the maximum inside the bin, the lowest
 * position winning ties (so an all-equal bin gives 0);
 * code = sum_k pos_k << (k * log2(bin)).
 * Densification (the "D" of DWTA, Section 4.1 names it only; reading, used
 * for queries when the flag is set): a bin of a query whose values are all
 * zero carries no information, so function p borrows the position of another
 * function's bin: it probes the functions p + 1 + (rng(seed, STREAM_PROBE,
 * r, p * DENSIFY_ATTEMPTS + a) mod (K*L - 1)) (mod K*L), a = 0, 1, ...,
 * DENSIFY_ATTEMPTS - 1, and takes the position of the first one whose own bin
 * is not all zero (never a borrowed one); when every probe fails, 0. */
static int dwta_position(const orc *o, const REAL *v, int p, int *all_zero) {
  const int bs = o->c.bin_size;
  const int32_t *idx = o->hash_idx + (size_t)p * bs;
  int best = 0, zero = 1;
  for (int i = 0; i < bs; ++i) {
    if (v[idx[i]] != 0) zero = 0;
    if (i >= 1 && v[idx[i]] > v[idx[best]]) best = i;
  }
  *all_zero = zero;
  return best;
}

static void hash_vec(const orc *o, const REAL *v, uint32_t *codes, int is_query) {
  const orc_config *c = &o->c;
  const int KL = c->K * c->L;
  for (int t = 0; t < c->L; ++t) {
    uint32_t code = 0;
    for (int k = 0; k < c->K; ++k) {
      int p = t * c->K + k;
      if (c->family == 0) {
        int m = c->srp_nnz;
        REAL s = 0;
        for (int i = 0; i < m; ++i) {
          REAL x = v[o->hash_idx[(size_t)p * m + i]];
          s = s + (o->hash_sign[(size_t)p * m + i] > 0 ? x : -x);
        }
        if (s >= 0) code |= 1u << k;
      } else {
        int bs = c->bin_size, lg = 0;
        while ((1 << lg) < bs) ++lg;
        int zero;
        int best = dwta_position(o, v, p, &zero);
        if (zero && is_query && c->densify && KL > 1) {
          best = 0;
          for (int a = 0; a < DENSIFY_ATTEMPTS; ++a) {
            uint64_t u = orc_rng(c->seed, STREAM_PROBE, (uint64_t)o->r, (uint64_t)p * DENSIFY_ATTEMPTS + (uint64_t)a);
            int g = (int)(((uint64_t)p + 1u + u % (uint64_t)(KL - 1)) % (uint64_t)KL);
            int gz;
            int gb = dwta_position(o, v, g, &gz);
            if (!gz) { best = gb; break; }
          }
        }
        code |= (uint32_t)best << (k * lg);
      }
    }
    codes[t] = code;
  }
}

/* codes of a neuron's weight row */
void orc_hash_vec(const orc *o, const REAL *v, uint32_t *codes) { hash_vec(o, v, codes, 0); }
/* codes of a query (a hidden activation) */
void orc_hash_query(const orc *o, const REAL *v, uint32_t *codes) { hash_vec(o, v, codes, 1); }

/* Section 2.1 phase 1 / Algorithm 1 "Hash weights to hash tables":
 * bucket (t, code) lists, in ascending id, every neuron whose weight row has
 * that code in table t. */
void orc_build_tables(orc *o) {
  const orc_config *c = &o->c;
  int64_t nb = (int64_t)1 << o->bits;
  uint32_t *codes = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)c->N * (size_t)c->L);
#pragma omp parallel for schedule(static)
  for (int j = 0; j < c->N; ++j) orc_hash_vec(o, o->W2 + (size_t)j * c->H, codes + (size_t)j * c->L);
#pragma omp parallel for schedule(dynamic, 1)
  for (int t = 0; t < c->L; ++t) {
    int32_t *cursor = (int32_t *)malloc(sizeof(int32_t) * (size_t)nb);
    int32_t *off = o->bucket_off + (size_t)t * (size_t)(nb + 1);
    int32_t *ids = o->bucket_ids + (size_t)t * (size_t)c->N;
    memset(off, 0, sizeof(int32_t) * (size_t)(nb + 1));
    for (int j = 0; j < c->N; ++j) off[codes[(size_t)j * c->L + t] + 1]++;
    for (int64_t b = 0; b < nb; ++b) off[b + 1] += off[b];
    for (int64_t b = 0; b < nb; ++b) cursor[b] = off[b];
    for (int j = 0; j < c->N; ++j) ids[cursor[codes[(size_t)j * c->L + t]]++] = j;
    free(cursor);
  }
  free(codes);
}

/* An unscheduled rebuild: next rebuild count, new functions if asked, tables. */
void orc_build_tables1(orc *o);
void orc_draw_hash1(orc *o, int64_t r);
void orc_rebuild_tables(orc *o) {
  o->r += 1;
  if (o->c.redraw) { orc_draw_hash(o, o->r); orc_draw_hash1(o, o->r); }
  orc_build_tables(o);
  orc_build_tables1(o);
}

/* ------------------------------------------------------------------ */
/* LSH-sampled hidden layer.                                           */
/* Hash family, reading: sparse random projections in their classic    */
/* form -- every entry of a projection is drawn by itself: +1 with     */
/* probability 1/6, -1 with probability 1/6, 0 with probability 2/3    */
/* (density 1/3, as for the output layer).  Entry (c, p) of rebuild    */
/* count r: u = rng(seed, STREAM_HASH1, r, c * KL + p); u mod 6 == 0   */
/* -> +1, == 1 -> -1, else 0.  (The output layer's projections choose   */
/* exactly ceil(H/3) coordinates by a shuffle; over the D input         */
/* coordinates a shuffle per projection is no plain definition any     */
/* more.)  Code of a vector v[D]: s_p = sum over the coordinates c of   */
/* the projection, ascending, of +-v[c], sequential in REAL;           */
/* bit = (s_p >= 0); code_t = sum_k bit_{tK+k} << k.                    */
/* ------------------------------------------------------------------ */
void orc_draw_hash1(orc *o, int64_t r) {
  const orc_config *c = &o->c;
  if (c->hidden_L <= 0) return;
  int64_t KL = (int64_t)c->hidden_K * c->hidden_L;
#pragma omp parallel for schedule(static)
  for (int64_t cc = 0; cc < c->D; ++cc)
    for (int64_t p = 0; p < KL; ++p) {
      uint64_t u = orc_rng(c->seed, STREAM_HASH1, (uint64_t)r, (uint64_t)cc * (uint64_t)KL + (uint64_t)p) % 6u;
      o->proj1[cc * KL + p] = u == 0 ? 1 : (u == 1 ? -1 : 0);
    }
}

/* codes of the sparse vector with nonzeros (col[j], val[j]), ascending columns: coordinates outside the vector add
 * nothing, so the sum over the projection's coordinates is the sum over the vector's nonzeros that it selects */
static void hash1_sparse(const orc *o, int32_t nnz, const int32_t *col, const REAL *val, uint32_t *codes) {
  const orc_config *c = &o->c;
  int64_t KL = (int64_t)c->hidden_K * c->hidden_L;
  for (int t = 0; t < c->hidden_L; ++t) {
    uint32_t code = 0;
    for (int k = 0; k < c->hidden_K; ++k) {
      int64_t p = (int64_t)t * c->hidden_K + k;
      REAL s = 0;
      for (int32_t j = 0; j < nnz; ++j) {
        int8_t e = o->proj1[(int64_t)col[j] * KL + p];
        if (e != 0) s = s + (e > 0 ? val[j] : -val[j]);
      }
      if (s >= 0) code |= 1u << k;
    }
    codes[t] = code;
  }
}

/* codes of hidden neuron k: its weight vector is column k of W1 */
static void hash1_neuron(const orc *o, int k, uint32_t *codes) {
  const orc_config *c = &o->c;
  int64_t KL = (int64_t)c->hidden_K * c->hidden_L;
  for (int t = 0; t < c->hidden_L; ++t) {
    uint32_t code = 0;
    for (int q = 0; q < c->hidden_K; ++q) {
      int64_t p = (int64_t)t * c->hidden_K + q;
      REAL s = 0;
      for (int64_t cc = 0; cc < c->D; ++cc) {
        int8_t e = o->proj1[cc * KL + p];
        if (e != 0) { REAL w = o->W1[(size_t)cc * c->H + k]; s = s + (e > 0 ? w : -w); }
      }
      if (s >= 0) code |= 1u << q;
    }
    codes[t] = code;
  }
}

/* tables over the hidden neurons: bucket (t, code) lists, ascending, the neurons with that code in table t */
void orc_build_tables1(orc *o) {
  const orc_config *c = &o->c;
  if (c->hidden_L <= 0) return;
  int64_t nb = (int64_t)1 << c->hidden_K;
  uint32_t *codes = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)c->H * (size_t)c->hidden_L);
#pragma omp parallel for schedule(dynamic, 1)
  for (int k = 0; k < c->H; ++k) hash1_neuron(o, k, codes + (size_t)k * c->hidden_L);
  for (int t = 0; t < c->hidden_L; ++t) {
    int32_t *off = o->bucket1_off + (size_t)t * (size_t)(nb + 1);
    int32_t *ids = o->bucket1_ids + (size_t)t * (size_t)c->H;
    memset(off, 0, sizeof(int32_t) * (size_t)(nb + 1));
    for (int k = 0; k < c->H; ++k) off[codes[(size_t)k * c->hidden_L + t] + 1]++;
    for (int64_t b = 0; b < nb; ++b) off[b + 1] += off[b];
    int32_t *cursor = (int32_t *)malloc(sizeof(int32_t) * (size_t)nb);
    for (int64_t b = 0; b < nb; ++b) cursor[b] = off[b];
    for (int k = 0; k < c->H; ++k) ids[cursor[codes[(size_t)k * c->hidden_L + t]]++] = k;
    free(cursor);
  }
  free(codes);
}

/* active hidden neurons of one sample: union over the tables of (at most hidden_cap lowest ids of) the buckets its
 * codes select; act[k] = 1 for an active neuron */
static void select_hidden(const orc *o, const uint32_t *codes, uint8_t *act) {
  const orc_config *c = &o->c;
  int64_t nb = (int64_t)1 << c->hidden_K;
  memset(act, 0, (size_t)c->H);
  for (int t = 0; t < c->hidden_L; ++t) {
    const int32_t *off = o->bucket1_off + (size_t)t * (size_t)(nb + 1);
    const int32_t *ids = o->bucket1_ids + (size_t)t * (size_t)c->H;
    int32_t cnt = off[codes[t] + 1] - off[codes[t]];
    if (cnt > c->hidden_cap) cnt = c->hidden_cap;
    for (int32_t i = 0; i < cnt; ++i) act[ids[off[codes[t]] + i]] = 1;
  }
}

static REAL *zalloc_real(int64_t n) { return (REAL *)calloc((size_t)(n > 0 ? n : 1), sizeof(REAL)); }

orc *orc_create(const orc_config *cfg) {
  orc *o = (orc *)calloc(1, sizeof(orc));
  o->c = *cfg;
  orc_config *c = &o->c;
  if (c->family == 0) {
    if (c->srp_nnz <= 0) c->srp_nnz = (c->H + 2) / 3;
    o->bits = c->K;
    o->idx_per_fn = c->srp_nnz;
  } else {
    int lg = 0;
    while ((1 << lg) < c->bin_size) ++lg;
    o->bits = c->K * lg;
    o->idx_per_fn = c->bin_size;
  }
  int64_t D = c->D, H = c->H, N = c->N;
  o->W1 = zalloc_real(D * H); o->mW1 = zalloc_real(D * H); o->vW1 = zalloc_real(D * H); o->dW1 = zalloc_real(D * H);
  o->b1 = zalloc_real(H); o->mb1 = zalloc_real(H); o->vb1 = zalloc_real(H); o->db1 = zalloc_real(H);
  o->W2 = zalloc_real(N * H); o->mW2 = zalloc_real(N * H); o->vW2 = zalloc_real(N * H); o->dW2 = zalloc_real(N * H);
  o->b2 = zalloc_real(N); o->mb2 = zalloc_real(N); o->vb2 = zalloc_real(N); o->db2 = zalloc_real(N);
  o->touch1 = (uint8_t *)calloc((size_t)D, 1);
  o->touch2 = (uint8_t *)calloc((size_t)N, 1);
  init_gauss(o->W1, D * H, c->seed, STREAM_W1, c->init_std);
  init_gauss(o->W2, N * H, c->seed, STREAM_W2, c->init_std);
  int64_t KL = (int64_t)c->K * c->L;
  o->hash_idx = (int32_t *)calloc((size_t)(KL * o->idx_per_fn), sizeof(int32_t));
  o->hash_sign = (int32_t *)calloc((size_t)(KL * o->idx_per_fn), sizeof(int32_t));
  int64_t nb = (int64_t)1 << o->bits;
  o->bucket_off = (int32_t *)calloc((size_t)(c->L * (nb + 1)), sizeof(int32_t));
  o->bucket_ids = (int32_t *)calloc((size_t)((int64_t)c->L * N), sizeof(int32_t));
  if (c->hidden_L > 0) {
    int64_t KL1 = (int64_t)c->hidden_K * c->hidden_L, nb1 = (int64_t)1 << c->hidden_K;
    o->proj1 = (int8_t *)calloc((size_t)(D * KL1), 1);
    o->bucket1_off = (int32_t *)calloc((size_t)(c->hidden_L * (nb1 + 1)), sizeof(int32_t));
    o->bucket1_ids = (int32_t *)calloc((size_t)((int64_t)c->hidden_L * H), sizeof(int32_t));
    o->touch1e = (uint8_t *)calloc((size_t)(D * H), 1);
  }
  o->t = 0; o->r = 0;
  o->next_rebuild = c->rebuild_period0;
  orc_draw_hash(o, 0);
  orc_build_tables(o);
  orc_draw_hash1(o, 0);
  orc_build_tables1(o);
  return o;
}

void orc_destroy(orc *o) {
  if (!o) return;
  free(o->W1); free(o->b1); free(o->W2); free(o->b2);
  free(o->mW1); free(o->vW1); free(o->mb1); free(o->vb1);
  free(o->mW2); free(o->vW2); free(o->mb2); free(o->vb2);
  free(o->dW1); free(o->db1); free(o->dW2); free(o->db2);
  free(o->touch1); free(o->touch2);
  free(o->hash_idx); free(o->hash_sign); free(o->bucket_off); free(o->bucket_ids);
  free(o->h); free(o->dh); free(o->codes); free(o->act_ptr); free(o->act_ids);
  free(o->act_z); free(o->act_p); free(o->act_g); free(o->loss);
  free(o->row_ptr); free(o->col_idx); free(o->vals); free(o->label_ptr); free(o->labels);
  free(o->proj1); free(o->bucket1_off); free(o->bucket1_ids); free(o->codes1); free(o->hact); free(o->touch1e);
  free(o);
}

static void ensure_batch(orc *o, int32_t B, int64_t nnz, int64_t nlab) {
  if (B > o->B_capacity) {
    int64_t H = o->c.H, L = o->c.L;
    o->h = (REAL *)realloc(o->h, sizeof(REAL) * (size_t)(B * H));
    o->dh = (REAL *)realloc(o->dh, sizeof(REAL) * (size_t)(B * H));
    o->codes = (uint32_t *)realloc(o->codes, sizeof(uint32_t) * (size_t)(B * L));
    o->act_ptr = (int64_t *)realloc(o->act_ptr, sizeof(int64_t) * (size_t)(B + 1));
    o->loss = (REAL *)realloc(o->loss, sizeof(REAL) * (size_t)B);
    o->row_ptr = (int32_t *)realloc(o->row_ptr, sizeof(int32_t) * (size_t)(B + 1));
    o->label_ptr = (int32_t *)realloc(o->label_ptr, sizeof(int32_t) * (size_t)(B + 1));
    if (o->c.hidden_L > 0) {
      o->codes1 = (uint32_t *)realloc(o->codes1, sizeof(uint32_t) * (size_t)(B * o->c.hidden_L));
      o->hact = (uint8_t *)realloc(o->hact, (size_t)(B * H));
    }
    o->B_capacity = B;
  }
  if (nnz > o->nnz_capacity) {
    o->col_idx = (int32_t *)realloc(o->col_idx, sizeof(int32_t) * (size_t)nnz);
    o->vals = (REAL *)realloc(o->vals, sizeof(REAL) * (size_t)nnz);
    o->nnz_capacity = nnz;
  }
  if (nlab > o->lab_capacity) {
    o->labels = (int32_t *)realloc(o->labels, sizeof(int32_t) * (size_t)nlab);
    o->lab_capacity = nlab;
  }
}

static void ensure_act(orc *o, int64_t need) {
  if (need <= o->act_capacity) return;
  int64_t cap = o->act_capacity ? o->act_capacity : 1024;
  while (cap < need) cap *= 2;
  o->act_ids = (int32_t *)realloc(o->act_ids, sizeof(int32_t) * (size_t)cap);
  o->act_z = (REAL *)realloc(o->act_z, sizeof(REAL) * (size_t)cap);
  o->act_p = (REAL *)realloc(o->act_p, sizeof(REAL) * (size_t)cap);
  o->act_g = (REAL *)realloc(o->act_g, sizeof(REAL) * (size_t)cap);
  o->act_capacity = cap;
}

/* Section 3.6, feed forward of the first type (sparse dataset input):
 * reading: bias first, then one fused multiply-add per nonzero in stored
 * order, then ReLU.  The order is part of the definition so that the hidden
 * activation, and with it every hash code, has one correct value. */
static void hidden_layer(const orc *o, int32_t nnz, const int32_t *col, const REAL *val, REAL *h, const uint8_t *act) {
  int H = o->c.H;
  for (int k = 0; k < H; ++k) {
    if (act && !act[k]) { h[k] = 0; continue; }     /* Section 2.1: a neuron that was not retrieved is a NoOp, activation 0 */
    REAL acc = o->b1[k];
    for (int32_t j = 0; j < nnz; ++j) acc = r_fma(val[j], o->W1[(size_t)col[j] * H + k], acc);
    h[k] = acc > 0 ? acc : 0;
  }
}

/* Is id one of the sample's labels? */
static int is_label(int32_t id, const int32_t *lab, int32_t nlab) {
  for (int32_t i = 0; i < nlab; ++i) if (lab[i] == id) return 1;
  return 0;
}

/* Section 3.7, the other option for a set below the budget: "fill the rest of
 * the sampling budget with uniformly sampled neurons".  reading: neurons are
 * drawn one after the other, id_k = rng(seed, STREAM_FILL, steps taken so
 * far, sample * 2^32 + k) mod N, k = 0, 1, ...; a draw that is already in the
 * set (retrieved, label, or drawn before) is passed over; drawing stops when
 * the set has min(budget, N) members or after 2 * (missing members) + 64
 * draws.  act[] must have room for budget entries; it is returned ascending. */
static int64_t fill_budget(const orc *o, int32_t *act, int64_t n, int32_t s) {
  const orc_config *c = &o->c;
  int64_t target = c->budget < c->N ? c->budget : c->N;
  if (n >= target) return n;
  int64_t need = target - n, draws = 2 * need + 64, got = 0;
  for (int64_t k = 0; k < draws && got < need; ++k) {
    uint64_t u = orc_rng(c->seed, STREAM_FILL, (uint64_t)o->t, ((uint64_t)(uint32_t)s << 32) + (uint64_t)k);
    int32_t id = (int32_t)(u % (uint64_t)c->N);
    int seen = 0;
    for (int64_t a = 0; a < n + got; ++a) if (act[a] == id) { seen = 1; break; }
    if (!seen) act[n + got++] = id;
  }
  qsort(act, (size_t)(n + got), sizeof(int32_t), cmp_i32);
  return n + got;
}

/* Section 3.7: when the neurons retrieved for a sample exceed the sampling
 * budget, reservoir sampling controls how many are kept; when they do not,
 * reading: the set is left as it is (the paper's "stop with the current set
 * of neurons") unless budget_fill asks for the paper's other option, the
 * uniform random fill (fill_budget above).
 * reading: the budget counts the sample's labels, which are always active,
 * so m = max(0, budget - |Y|) of the other retrieved neurons are kept.  The
 * candidates C_0 < C_1 < ... (retrieved ids that are not labels, ascending)
 * go through the textbook reservoir algorithm: the first m fill the
 * reservoir; candidate i >= m draws j uniform in [0, i] and replaces
 * reservoir[j] when j < m.  j = rng(seed, STREAM_SAMPLE, steps taken so far,
 * sample * 2^32 + i) mod (i + 1).  act[] (ascending, n entries) is rewritten
 * with the labels and the reservoir, ascending; returns the new count. */
static int64_t apply_budget(const orc *o, int32_t *act, int64_t n, const int32_t *lab, int32_t nlab, int32_t s) {
  const orc_config *c = &o->c;
  int64_t ny = 0, nc = 0;
  for (int64_t a = 0; a < n; ++a) { if (is_label(act[a], lab, nlab)) ++ny; else ++nc; }
  int64_t m = c->budget - ny;
  if (m < 0) m = 0;
  if (nc <= m) return c->budget_fill ? fill_budget(o, act, n, s) : n;
  int32_t *cand = (int32_t *)malloc(sizeof(int32_t) * (size_t)(nc > 0 ? nc : 1));
  int32_t *res = (int32_t *)malloc(sizeof(int32_t) * (size_t)(m > 0 ? m : 1));
  int64_t k = 0;
  for (int64_t a = 0; a < n; ++a) if (!is_label(act[a], lab, nlab)) cand[k++] = act[a];
  for (int64_t i = 0; i < nc; ++i) {
    if (i < m) { res[i] = cand[i]; continue; }
    uint64_t u = orc_rng(c->seed, STREAM_SAMPLE, (uint64_t)o->t, ((uint64_t)(uint32_t)s << 32) + (uint64_t)i);
    uint64_t j = u % (uint64_t)(i + 1);
    if (j < (uint64_t)m) res[j] = cand[i];
  }
  int64_t out = 0;
  for (int64_t a = 0; a < n; ++a) if (is_label(act[a], lab, nlab)) act[out++] = act[a];
  for (int64_t j = 0; j < m; ++j) act[out++] = res[j];
  qsort(act, (size_t)out, sizeof(int32_t), cmp_i32);
  free(cand); free(res);
  return out;
}

/* Section 2.1 feed-forward stage + Fig. 1: query the L tables with the layer
 * input, take the union of the retrieved buckets (at most bucket_cap lowest
 * ids of each), add the labels when given (reading: labels are always
 * active), sort, remove duplicates, then apply the sampling budget when one
 * is set.  Returns the count. */
static int64_t select_active(const orc *o, const uint32_t *codes, const int32_t *lab, int32_t nlab,
                             int32_t **buf, int64_t *bufcap, int32_t s) {
  const orc_config *c = &o->c;
  int64_t n = 0;
  if (c->force_dense) {
    if (*bufcap < c->N) { *buf = (int32_t *)realloc(*buf, sizeof(int32_t) * (size_t)c->N); *bufcap = c->N; }
    for (int j = 0; j < c->N; ++j) (*buf)[j] = j;
    return c->N;
  }
  int64_t worst = (int64_t)c->L * c->bucket_cap + nlab;
  if (c->budget_fill && worst < c->budget) worst = c->budget;
  if (*bufcap < worst) { *buf = (int32_t *)realloc(*buf, sizeof(int32_t) * (size_t)worst); *bufcap = worst; }
  int64_t nb = (int64_t)1 << o->bits;
  for (int t = 0; t < c->L; ++t) {
    const int32_t *off = o->bucket_off + (size_t)t * (size_t)(nb + 1);
    const int32_t *ids = o->bucket_ids + (size_t)t * (size_t)c->N;
    int32_t cnt = off[codes[t] + 1] - off[codes[t]];
    if (cnt > c->bucket_cap) cnt = c->bucket_cap;
    for (int32_t i = 0; i < cnt; ++i) (*buf)[n++] = ids[off[codes[t]] + i];
  }
  for (int32_t i = 0; i < nlab; ++i) (*buf)[n++] = lab[i];
  qsort(*buf, (size_t)n, sizeof(int32_t), cmp_i32);
  int64_t u = 0;
  for (int64_t i = 0; i < n; ++i)
    if (u == 0 || (*buf)[u - 1] != (*buf)[i]) (*buf)[u++] = (*buf)[i];
  if (c->budget > 0) u = apply_budget(o, *buf, u, lab, nlab, s);
  return u;
}

/* One forward pass over a batch (Algorithm 1 inner loops: retrieve active
 * neurons, feed forward, compute errors).  Labels may be NULL (inference).
 * reading (loss): softmax over the active set only, cross-entropy against
 * the uniform distribution over the sample's distinct labels; the error of
 * neuron j is (p_j - [j in Y]/|Y|) / B (mean over the batch). */
int32_t orc_forward(orc *o, int32_t B, const int32_t *row_ptr, const int32_t *col_idx, const REAL *vals,
                    const int32_t *label_ptr, const int32_t *labels) {
  const orc_config *c = &o->c;
  int H = c->H;
  int64_t nnz = row_ptr[B], nlab = label_ptr ? label_ptr[B] : 0;
  ensure_batch(o, B, nnz, nlab);
  o->B = B;
  o->error = 0;
  memcpy(o->row_ptr, row_ptr, sizeof(int32_t) * (size_t)(B + 1));
  memcpy(o->col_idx, col_idx, sizeof(int32_t) * (size_t)nnz);
  memcpy(o->vals, vals, sizeof(REAL) * (size_t)nnz);
  if (label_ptr) {
    memcpy(o->label_ptr, label_ptr, sizeof(int32_t) * (size_t)(B + 1));
    memcpy(o->labels, labels, sizeof(int32_t) * (size_t)nlab);
  }
  for (int64_t i = 0; i < nnz; ++i)
    if (col_idx[i] < 0 || col_idx[i] >= c->D) { o->error = 5; return o->error; }
  for (int64_t i = 0; i < nlab; ++i)
    if (labels[i] < 0 || labels[i] >= c->N) { o->error = 5; return o->error; }

  /* first loop over the samples: hidden activation, codes, active set (kept per sample) */
  int32_t **sel = (int32_t **)calloc((size_t)B, sizeof(int32_t *));
  int64_t *na_of = (int64_t *)calloc((size_t)B, sizeof(int64_t));
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t s = 0; s < B; ++s) {
    REAL *h = o->h + (size_t)s * H;
    const uint8_t *hact = NULL;
    if (c->hidden_L > 0) {      /* Algorithm 1: retrieve the layer's active neurons with the layer's input, then feed forward */
      uint32_t *codes1 = o->codes1 + (size_t)s * c->hidden_L;
      hash1_sparse(o, row_ptr[s + 1] - row_ptr[s], col_idx + row_ptr[s], vals + row_ptr[s], codes1);
      select_hidden(o, codes1, o->hact + (size_t)s * H);
      hact = o->hact + (size_t)s * H;
    }
    hidden_layer(o, row_ptr[s + 1] - row_ptr[s], col_idx + row_ptr[s], vals + row_ptr[s], h, hact);
    uint32_t *codes = o->codes + (size_t)s * c->L;
    orc_hash_query(o, h, codes);
    const int32_t *lab = label_ptr ? labels + label_ptr[s] : NULL;
    int32_t nl = label_ptr ? label_ptr[s + 1] - label_ptr[s] : 0;
    int32_t *buf = NULL; int64_t bufcap = 0;
    na_of[s] = select_active(o, codes, lab, nl, &buf, &bufcap, s);
    sel[s] = buf;
  }
  /* where each sample's entries go in the snapshot arrays */
  o->act_ptr[0] = 0;
  for (int32_t s = 0; s < B; ++s) {
    if (c->max_active > 0 && na_of[s] > c->max_active) o->error = 4;
    o->act_ptr[s + 1] = o->act_ptr[s] + na_of[s];
  }
  if (o->error) {
    for (int32_t s = 0; s < B; ++s) free(sel[s]);
    free(sel); free(na_of);
    return o->error;
  }
  ensure_act(o, o->act_ptr[B]);
  /* second loop over the samples: activations of the active neurons, softmax, errors */
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t s = 0; s < B; ++s) {
    const REAL *h = o->h + (size_t)s * H;
    const int32_t *buf = sel[s];
    const int32_t *lab = label_ptr ? labels + label_ptr[s] : NULL;
    int32_t nl = label_ptr ? label_ptr[s + 1] - label_ptr[s] : 0;
    int64_t base = o->act_ptr[s], na = na_of[s];
    memcpy(o->act_ids + base, buf, sizeof(int32_t) * (size_t)na);

    /* feed forward of the second type over the active neurons only (Section 3.6) */
    REAL *z = o->act_z + base, *p = o->act_p + base, *g = o->act_g + base;
    for (int64_t a = 0; a < na; ++a) {
      int32_t j = buf[a];
      REAL acc = 0;
      for (int k = 0; k < H; ++k) acc += o->W2[(size_t)j * H + k] * h[k];
      z[a] = o->b2[j] + acc;
    }
    /* softmax over the active set */
    REAL M = z[0];
    for (int64_t a = 1; a < na; ++a) if (z[a] > M) M = z[a];
    REAL E = 0;
    for (int64_t a = 0; a < na; ++a) { p[a] = r_exp(z[a] - M); E += p[a]; }
    for (int64_t a = 0; a < na; ++a) p[a] = p[a] / E;
    /* errors (Algorithm 1 "Compute Errors") */
    o->loss[s] = 0;
    for (int64_t a = 0; a < na; ++a) g[a] = p[a];
    if (label_ptr) {
      /* distinct labels of this sample */
      int32_t ny = 0;
      for (int64_t a = 0; a < na; ++a) {
        int is_label = 0;
        for (int32_t i = 0; i < nl; ++i) if (lab[i] == buf[a]) { is_label = 1; break; }
        if (is_label) ++ny;
      }
      REAL logE = r_log(E), sum = 0;
      for (int64_t a = 0; a < na; ++a) {
        int is_label = 0;
        for (int32_t i = 0; i < nl; ++i) if (lab[i] == buf[a]) { is_label = 1; break; }
        if (is_label) { sum += z[a] - M - logE; g[a] = p[a] - (REAL)1 / (REAL)ny; }
      }
      o->loss[s] = ny > 0 ? -sum / (REAL)ny : 0;
    }
    for (int64_t a = 0; a < na; ++a) g[a] = g[a] / (REAL)B;
  }
  for (int32_t s = 0; s < B; ++s) free(sel[s]);
  free(sel); free(na_of);
  return 0;
}

/* Section 2.1 back-propagation stage: errors and gradients reach the active
 * neurons only.  Uses the weights as they were in the forward pass.
 * Gradients are summed over the samples in ascending order. */
void orc_backward(orc *o) {
  const orc_config *c = &o->c;
  int H = c->H;
  /* error at the hidden layer, sample by sample */
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t s = 0; s < o->B; ++s) {
    const REAL *h = o->h + (size_t)s * H;
    REAL *dh = o->dh + (size_t)s * H;
    for (int k = 0; k < H; ++k) dh[k] = 0;
    for (int64_t a = o->act_ptr[s]; a < o->act_ptr[s + 1]; ++a) {
      int32_t j = o->act_ids[a];
      REAL g = o->act_g[a];
      for (int k = 0; k < H; ++k) dh[k] += g * o->W2[(size_t)j * H + k];
    }
    for (int k = 0; k < H; ++k) if (!(h[k] > 0)) dh[k] = 0;   /* ReLU derivative */
  }
  /* gradients of the rows, samples in ascending order; a worker adds only into the rows it owns */
#pragma omp parallel
  {
    int tid, nt;
    who_am_i(&tid, &nt);
    for (int32_t s = 0; s < o->B; ++s) {
      const REAL *h = o->h + (size_t)s * H;
      const REAL *dh = o->dh + (size_t)s * H;
      for (int64_t a = o->act_ptr[s]; a < o->act_ptr[s + 1]; ++a) {
        int32_t j = o->act_ids[a];
        if (j % nt != tid) continue;
        REAL g = o->act_g[a];
        for (int k = 0; k < H; ++k) o->dW2[(size_t)j * H + k] += g * h[k];
        o->db2[j] += g;
        o->touch2[j] = 1;
      }
      for (int32_t i = o->row_ptr[s]; i < o->row_ptr[s + 1]; ++i) {
        int32_t f = o->col_idx[i];
        if (f % nt != tid) continue;
        REAL x = o->vals[i];
        for (int k = 0; k < H; ++k) o->dW1[(size_t)f * H + k] += x * dh[k];
        o->touch1[f] = 1;
        if (o->touch1e) {     /* sampled hidden layer: only the weights of the sample's active hidden neurons are touched */
          const uint8_t *hact = o->hact + (size_t)s * H;
          for (int k = 0; k < H; ++k) if (hact[k]) o->touch1e[(size_t)f * H + k] = 1;
        }
      }
      for (int k = tid; k < H; k += nt) o->db1[k] += dh[k];
    }
  }
}

static void adam_elem(const orc *o, REAL *w, REAL *m, REAL *v, REAL g, REAL bc1, REAL bc2) {
  REAL b1 = (REAL)o->c.beta1, b2 = (REAL)o->c.beta2;
  *m = b1 * (*m) + ((REAL)1 - b1) * g;
  *v = b2 * (*v) + ((REAL)1 - b2) * g * g;
  REAL mhat = *m / bc1, vhat = *v / bc2;
  *w = *w - (REAL)o->c.lr * mhat / (r_sqrt(vhat) + (REAL)o->c.eps);
}

/* Algorithm 1 "Update weights with Adam" (constants: Section 4.1; a momentum
 * and a velocity array per weight and per bias array: Section 3.5).
 * reading: only rows touched by this batch are updated (and the dense hidden
 * bias); untouched rows keep weight and moments unchanged; the bias
 * correction uses the global step count.  Clears the gradient buffers. */
void orc_adam(orc *o) {
  const orc_config *c = &o->c;
  int H = c->H;
  o->t += 1;
  REAL bc1 = (REAL)(1.0 - pow(c->beta1, (double)o->t));
  REAL bc2 = (REAL)(1.0 - pow(c->beta2, (double)o->t));
#pragma omp parallel for schedule(static)
  for (int j = 0; j < c->N; ++j) {
    if (!o->touch2[j]) continue;
    for (int k = 0; k < H; ++k) {
      size_t e = (size_t)j * H + k;
      adam_elem(o, &o->W2[e], &o->mW2[e], &o->vW2[e], o->dW2[e], bc1, bc2);
      o->dW2[e] = 0;
    }
    adam_elem(o, &o->b2[j], &o->mb2[j], &o->vb2[j], o->db2[j], bc1, bc2);
    o->db2[j] = 0;
    o->touch2[j] = 0;
  }
#pragma omp parallel for schedule(static)
  for (int f = 0; f < c->D; ++f) {
    if (!o->touch1[f]) continue;
    for (int k = 0; k < H; ++k) {
      size_t e = (size_t)f * H + k;
      if (!o->touch1e || o->touch1e[e]) adam_elem(o, &o->W1[e], &o->mW1[e], &o->vW1[e], o->dW1[e], bc1, bc2);
      if (o->touch1e) o->touch1e[e] = 0;
      o->dW1[e] = 0;
    }
    o->touch1[f] = 0;
  }
  for (int k = 0; k < H; ++k) {
    /* a sampled hidden layer: the bias of a neuron that no sample of the batch retrieved is untouched */
    int touched = 1;
    if (c->hidden_L > 0) {
      touched = 0;
      for (int32_t s = 0; s < o->B; ++s) if (o->hact[(size_t)s * H + k]) { touched = 1; break; }
    }
    if (touched) adam_elem(o, &o->b1[k], &o->mb1[k], &o->vb1[k], o->db1[k], bc1, bc2);
    o->db1[k] = 0;
  }
}

/* Rebuild schedule (Section 3.1 "locally updated with a frequency schedule";
 * Algorithm 1 places the rebuild after the weight update).
 * reading: first rebuild after p0 steps, then gaps max(1, floor(p0*exp(lambda*r))). */
int32_t orc_schedule(orc *o) {
  if (o->c.rebuild_period0 <= 0 || o->t != o->next_rebuild) return 0;
  orc_rebuild_tables(o);
  double gap = floor((double)o->c.rebuild_period0 * exp(o->c.rebuild_lambda * (double)o->r));
  if (gap < 1.0) gap = 1.0;
  o->next_rebuild += (int64_t)gap;
  return 1;
}

/* One full training step on one batch; returns the mean loss through *loss_out. */
int32_t orc_train_step(orc *o, int32_t B, const int32_t *row_ptr, const int32_t *col_idx, const REAL *vals,
                       const int32_t *label_ptr, const int32_t *labels, double *loss_out) {
  int32_t e = orc_forward(o, B, row_ptr, col_idx, vals, label_ptr, labels);
  if (e) return e;
  REAL sum = 0;
  for (int32_t s = 0; s < B; ++s) sum += o->loss[s];
  if (loss_out) *loss_out = (double)(sum / (REAL)B);
  orc_backward(o);
  orc_adam(o);
  orc_schedule(o);
  return 0;
}

/* Inference (the paper reports test accuracy but not how it evaluates;
 * reading: logits over the retrieved set, or over every neuron when dense,
 * then the k largest by (logit descending, id ascending); missing entries are
 * id -1 with score -infinity). */
int32_t orc_predict_topk(orc *o, int32_t B, const int32_t *row_ptr, const int32_t *col_idx, const REAL *vals,
                         int32_t k, int32_t dense, int32_t *out_ids, REAL *out_scores) {
  int32_t saved = o->c.force_dense;
  if (dense) o->c.force_dense = 1;
  int32_t e = orc_forward(o, B, row_ptr, col_idx, vals, NULL, NULL);
  o->c.force_dense = saved;
  if (e) return e;
  for (int32_t s = 0; s < B; ++s) {
    int64_t base = o->act_ptr[s], na = o->act_ptr[s + 1] - base;
    uint8_t *used = (uint8_t *)calloc((size_t)(na > 0 ? na : 1), 1);
    for (int32_t q = 0; q < k; ++q) {
      int64_t best = -1;
      for (int64_t a = 0; a < na; ++a) {
        if (used[a]) continue;
        if (best < 0 || o->act_z[base + a] > o->act_z[base + best]) best = a;   /* ids ascend, so ties keep the lower id */
      }
      if (best >= 0) {
        used[best] = 1;
        out_ids[(size_t)s * k + q] = o->act_ids[base + best];
        out_scores[(size_t)s * k + q] = o->act_z[base + best];
      } else {
        out_ids[(size_t)s * k + q] = -1;
        out_scores[(size_t)s * k + q] = (REAL)(-INFINITY);
      }
    }
    free(used);
  }
  return 0;
}

/* ------------------------------------------------------------------ */
/* Accessors for the Python test harness.                              */
/* ------------------------------------------------------------------ */
enum {
  ORC_W1 = 0, ORC_B1, ORC_W2, ORC_B2, ORC_MW1, ORC_VW1, ORC_MB1, ORC_VB1, ORC_MW2, ORC_VW2, ORC_MB2, ORC_VB2,
  ORC_DW1, ORC_DB1, ORC_DW2, ORC_DB2,
  ORC_HASH_IDX, ORC_HASH_SIGN, ORC_BUCKET_OFF, ORC_BUCKET_IDS,
  ORC_H, ORC_DH, ORC_CODES, ORC_ACT_PTR, ORC_ACT_IDS, ORC_ACT_Z, ORC_ACT_P, ORC_ACT_G, ORC_LOSS,
  ORC_PROJ1, ORC_BUCKET1_OFF, ORC_BUCKET1_IDS, ORC_CODES1, ORC_HACT
};

void *orc_ptr(orc *o, int32_t which) {
  switch (which) {
    case ORC_W1: return o->W1; case ORC_B1: return o->b1; case ORC_W2: return o->W2; case ORC_B2: return o->b2;
    case ORC_MW1: return o->mW1; case ORC_VW1: return o->vW1; case ORC_MB1: return o->mb1; case ORC_VB1: return o->vb1;
    case ORC_MW2: return o->mW2; case ORC_VW2: return o->vW2; case ORC_MB2: return o->mb2; case ORC_VB2: return o->vb2;
    case ORC_DW1: return o->dW1; case ORC_DB1: return o->db1; case ORC_DW2: return o->dW2; case ORC_DB2: return o->db2;
    case ORC_HASH_IDX: return o->hash_idx; case ORC_HASH_SIGN: return o->hash_sign;
    case ORC_BUCKET_OFF: return o->bucket_off; case ORC_BUCKET_IDS: return o->bucket_ids;
    case ORC_H: return o->h; case ORC_DH: return o->dh; case ORC_CODES: return o->codes;
    case ORC_ACT_PTR: return o->act_ptr; case ORC_ACT_IDS: return o->act_ids;
    case ORC_ACT_Z: return o->act_z; case ORC_ACT_P: return o->act_p; case ORC_ACT_G: return o->act_g;
    case ORC_LOSS: return o->loss;
    case ORC_PROJ1: return o->proj1; case ORC_BUCKET1_OFF: return o->bucket1_off; case ORC_BUCKET1_IDS: return o->bucket1_ids;
    case ORC_CODES1: return o->codes1; case ORC_HACT: return o->hact;
  }
  return NULL;
}

int64_t orc_count(orc *o, int32_t which) {
  const orc_config *c = &o->c;
  int64_t D = c->D, H = c->H, N = c->N, KL = (int64_t)c->K * c->L, nb = (int64_t)1 << o->bits;
  switch (which) {
    case ORC_W1: case ORC_MW1: case ORC_VW1: case ORC_DW1: return D * H;
    case ORC_B1: case ORC_MB1: case ORC_VB1: case ORC_DB1: return H;
    case ORC_W2: case ORC_MW2: case ORC_VW2: case ORC_DW2: return N * H;
    case ORC_B2: case ORC_MB2: case ORC_VB2: case ORC_DB2: return N;
    case ORC_HASH_IDX: return KL * o->idx_per_fn;
    case ORC_HASH_SIGN: return c->family == 0 ? KL * o->idx_per_fn : 0;
    case ORC_BUCKET_OFF: return c->L * (nb + 1);
    case ORC_BUCKET_IDS: return (int64_t)c->L * N;
    case ORC_H: case ORC_DH: return (int64_t)o->B * H;
    case ORC_CODES: return (int64_t)o->B * c->L;
    case ORC_ACT_PTR: return o->B + 1;
    case ORC_ACT_IDS: case ORC_ACT_Z: case ORC_ACT_P: case ORC_ACT_G: return o->B ? o->act_ptr[o->B] : 0;
    case ORC_LOSS: return o->B;
    case ORC_PROJ1: return c->hidden_L > 0 ? D * c->hidden_K * c->hidden_L : 0;
    case ORC_BUCKET1_OFF: return c->hidden_L > 0 ? c->hidden_L * (((int64_t)1 << c->hidden_K) + 1) : 0;
    case ORC_BUCKET1_IDS: return c->hidden_L > 0 ? (int64_t)c->hidden_L * H : 0;
    case ORC_CODES1: return c->hidden_L > 0 ? (int64_t)o->B * c->hidden_L : 0;
    case ORC_HACT: return c->hidden_L > 0 ? (int64_t)o->B * H : 0;
  }
  return -1;
}

int64_t orc_step_count(const orc *o) { return o->t; }
int64_t orc_rebuild_count(const orc *o) { return o->r; }
int64_t orc_next_rebuild(const orc *o) { return o->next_rebuild; }
void orc_set_counters(orc *o, int64_t t, int64_t r, int64_t next_rebuild) { o->t = t; o->r = r; o->next_rebuild = next_rebuild; }
int32_t orc_bits(const orc *o) { return o->bits; }
int32_t orc_idx_per_fn(const orc *o) { return o->idx_per_fn; }
int32_t orc_sizeof_real(void) { return (int32_t)sizeof(REAL); }
int32_t orc_last_error(const orc *o) { return o->error; }
