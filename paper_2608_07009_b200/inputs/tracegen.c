/*
 * Seeded synthetic inputs for the selection-resolution path: host KV-history bytes and
 * selection traces shaped like DSA (token level), NSA (block level) and Quest (page level)
 * decoding.  This file holds no cache arithmetic: it only draws inputs.  Both the CPU oracle's
 * tests and the CUDA path's tests/bench call it, so neither side's inputs depend on the other.
 *
 * Everything is a pure function of (seed, indices): a counter-based generator built on the
 * splitmix64 finaliser, so any record or any row can be regenerated alone.
 *
 * Plain C, no dependencies; built as a shared library and called through ctypes.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define GOLDEN 0x9E3779B97F4A7C15ull

static inline uint64_t mix64(uint64_t z) {
  z += GOLDEN;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

/* ------------------------------------------------------------------ history bytes */

static inline uint64_t record_key(uint64_t seed, int64_t r, int64_t l, int64_t pos) {
  uint64_t a = mix64(seed ^ 0x48695370617273ull); /* "HiSpars" */
  a = mix64(a + (uint64_t)r);
  a = mix64(a + (uint64_t)l);
  return mix64(a + (uint64_t)pos);
}

/* Bytes of record (r, l, pos): 8-byte word w is mix64(key + w*GOLDEN); a tail shorter than
 * 8 bytes takes the low bytes of its word.  entry_bytes may be any positive size. */
void hs_record_fill(uint8_t *dst, int64_t r, int64_t l, int64_t pos, int64_t entry_bytes,
                    uint64_t seed) {
  uint64_t key = record_key(seed, r, l, pos);
  int64_t w = 0, off = 0;
  for (; off + 8 <= entry_bytes; off += 8, ++w) {
    uint64_t v = mix64(key + (uint64_t)w * GOLDEN);
    memcpy(dst + off, &v, 8);
  }
  if (off < entry_bytes) {
    uint64_t v = mix64(key + (uint64_t)w * GOLDEN);
    memcpy(dst + off, &v, (size_t)(entry_bytes - off));
  }
}

typedef struct {
  uint8_t *base;
  int64_t r, L, cap, pos0, pos1, E;
  uint64_t seed;
  int tid, nthreads;
} fill_job_t;

static void *fill_worker(void *arg) {
  fill_job_t *j = (fill_job_t *)arg;
  int64_t npos = j->pos1 - j->pos0;
  int64_t total = j->L * npos;
  int64_t lo = total * j->tid / j->nthreads, hi = total * (j->tid + 1) / j->nthreads;
  for (int64_t i = lo; i < hi; ++i) {
    int64_t l = i / npos, pos = j->pos0 + i % npos;
    hs_record_fill(j->base + (l * j->cap + pos) * j->E, j->r, l, pos, j->E, j->seed);
  }
  return NULL;
}

/* Fill request r's history, laid out [L][cap][E], for positions pos0 <= pos < pos1 of every
 * layer, using up to `threads` threads. */
void hs_history_fill(uint8_t *base, int64_t r, int64_t L, int64_t cap, int64_t pos0, int64_t pos1,
                     int64_t entry_bytes, uint64_t seed, int threads) {
  if (threads < 1) threads = 1;
  if (threads > 64) threads = 64;
  pthread_t th[64];
  fill_job_t jobs[64];
  for (int t = 0; t < threads; ++t) {
    jobs[t] = (fill_job_t){base, r, L, cap, pos0, pos1, entry_bytes, seed, t, threads};
    if (t > 0) pthread_create(&th[t], NULL, fill_worker, &jobs[t]);
  }
  fill_worker(&jobs[0]);
  for (int t = 1; t < threads; ++t) pthread_join(th[t], NULL);
}

/* new_kv[N][L][E] for one append: request r appends position pos[r]. */
void hs_new_kv_fill(uint8_t *dst, int64_t N, int64_t L, const int64_t *pos, int64_t entry_bytes,
                    uint64_t seed) {
  for (int64_t r = 0; r < N; ++r)
    for (int64_t l = 0; l < L; ++l)
      hs_record_fill(dst + (r * L + l) * entry_bytes, r, l, pos[r], entry_bytes, seed);
}

/* ------------------------------------------------------------------ selection traces */

enum {
  HS_TRACE_DSA_ZIPF = 0, /* keep a fraction; redraw from Zipf over recency ranks         */
  HS_TRACE_DSA_MIX = 1,  /* keep a fraction; redraw half from a recent window, half uniform */
  HS_TRACE_NSA_BLOCKS = 2, /* k-2 blocks by Zipf over a fixed popularity order + 2 local blocks */
  HS_TRACE_QUEST_PAGES = 3 /* top-k pages of AR(1)-drifting Gaussian scores               */
};

typedef struct {
  int32_t kind;
  int32_t num_requests;   /* N */
  int32_t num_streams;    /* G: independent selection streams per request (anchor layers) */
  int32_t top_k;          /* k */
  int32_t append_every;   /* a record is appended at step s when (s+1) % append_every == 0 */
  int32_t recent_window;  /* DSA_MIX: width of the recent window                        */
  int32_t zipf_support;   /* DSA_ZIPF: number of recency ranks; NSA: popularity ranks   */
  int32_t keep;           /* rows entries kept from the previous step                   */
  double zipf_s;          /* Zipf exponent                                              */
  double ar_rho;          /* QUEST: AR(1) coefficient                                   */
  uint64_t seed;
  int32_t config_id;      /* mixed into every stream key                                */
} hs_trace_params_t;

typedef struct {
  uint64_t key, ctr;
} rng_t;

static inline uint64_t rng_u64(rng_t *g) { return mix64(g->key + (g->ctr++) * GOLDEN); }
static inline double rng_unit(rng_t *g) { return (double)(rng_u64(g) >> 11) * (1.0 / 9007199254740992.0); }
static inline int64_t rng_below(rng_t *g, int64_t n) { return (int64_t)(rng_u64(g) % (uint64_t)n); }
static double rng_gauss(rng_t *g) {
  double u1 = rng_unit(g), u2 = rng_unit(g);
  if (u1 < 1e-300) u1 = 1e-300;
  return sqrt(-2.0 * log(u1)) * cos(6.283185307179586 * u2);
}

typedef struct {
  rng_t rng;
  int32_t *row;      /* [k] current selection */
  uint8_t *member;   /* [cap] 1 if the position is in the row */
  double *score;     /* QUEST: [cap] */
  int32_t *perm;     /* NSA: popularity order of blocks */
  int32_t *idx;      /* [k] scratch */
  int started;
} stream_t;

typedef struct {
  hs_trace_params_t p;
  int64_t *len;      /* [N] current history length */
  int64_t *cap;      /* [N] */
  stream_t *st;      /* [N*G] */
  double *zipf_cdf;  /* [zipf_support] */
  int64_t step;
} hs_trace_t;

static int cmp_i32(const void *a, const void *b) {
  int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
  return (x > y) - (x < y);
}

static int64_t zipf_draw(const hs_trace_t *t, rng_t *g) {
  double u = rng_unit(g) * t->zipf_cdf[t->p.zipf_support - 1];
  int64_t lo = 0, hi = t->p.zipf_support - 1;
  while (lo < hi) {
    int64_t mid = (lo + hi) / 2;
    if (t->zipf_cdf[mid] > u) hi = mid; else lo = mid + 1;
  }
  return lo; /* rank - 1 */
}

hs_trace_t *hs_trace_create(const hs_trace_params_t *p, const int64_t *init_len, const int64_t *cap) {
  hs_trace_t *t = (hs_trace_t *)calloc(1, sizeof *t);
  t->p = *p;
  int N = p->num_requests, G = p->num_streams, k = p->top_k;
  t->len = (int64_t *)malloc(sizeof(int64_t) * N);
  t->cap = (int64_t *)malloc(sizeof(int64_t) * N);
  memcpy(t->len, init_len, sizeof(int64_t) * N);
  memcpy(t->cap, cap, sizeof(int64_t) * N);
  if (p->zipf_support > 0) {
    t->zipf_cdf = (double *)malloc(sizeof(double) * p->zipf_support);
    double acc = 0;
    for (int i = 0; i < p->zipf_support; ++i) { acc += pow((double)(i + 1), -p->zipf_s); t->zipf_cdf[i] = acc; }
  }
  t->st = (stream_t *)calloc((size_t)N * G, sizeof(stream_t));
  for (int r = 0; r < N; ++r)
    for (int g = 0; g < G; ++g) {
      stream_t *s = &t->st[r * G + g];
      uint64_t key = mix64(p->seed ^ 0x7472616365ull);
      key = mix64(key + (uint64_t)p->config_id);
      key = mix64(key + (uint64_t)r);
      key = mix64(key + (uint64_t)g);
      s->rng.key = key; s->rng.ctr = 0;
      s->row = (int32_t *)malloc(sizeof(int32_t) * k);
      s->idx = (int32_t *)malloc(sizeof(int32_t) * k);
      s->member = (uint8_t *)calloc((size_t)cap[r], 1);
      for (int j = 0; j < k; ++j) s->row[j] = -1;
      if (p->kind == HS_TRACE_QUEST_PAGES) {
        s->score = (double *)malloc(sizeof(double) * cap[r]);
        for (int64_t q = 0; q < init_len[r]; ++q) s->score[q] = rng_gauss(&s->rng);
      }
      if (p->kind == HS_TRACE_NSA_BLOCKS) {
        int n = p->zipf_support;
        s->perm = (int32_t *)malloc(sizeof(int32_t) * n);
        for (int i = 0; i < n; ++i) s->perm[i] = i;
        for (int i = n - 1; i > 0; --i) {
          int j = (int)rng_below(&s->rng, i + 1);
          int32_t tmp = s->perm[i]; s->perm[i] = s->perm[j]; s->perm[j] = tmp;
        }
      }
    }
  return t;
}

void hs_trace_destroy(hs_trace_t *t) {
  if (!t) return;
  int n = t->p.num_requests * t->p.num_streams;
  for (int i = 0; i < n; ++i) {
    free(t->st[i].row); free(t->st[i].idx); free(t->st[i].member); free(t->st[i].score); free(t->st[i].perm);
  }
  free(t->st); free(t->len); free(t->cap); free(t->zipf_cdf); free(t);
}

/* A position not yet in the row: first the class's own distribution (<= 64 tries), then uniform
 * over the history (<= 64 tries), then the first free position after a random start. */
static int32_t draw_distinct(hs_trace_t *t, stream_t *s, int64_t len, int cls, int64_t lo_allowed,
                             int64_t hi_allowed) {
  const hs_trace_params_t *p = &t->p;
  for (int tries = 0; tries < 64; ++tries) {
    int64_t pos;
    if (cls == 0) { /* Zipf over recency rank: rank 1 is the newest position */
      pos = len - 1 - zipf_draw(t, &s->rng);
    } else if (cls == 1) { /* uniform over the recent window */
      int64_t w = p->recent_window < len ? p->recent_window : len;
      pos = len - 1 - rng_below(&s->rng, w);
    } else if (cls == 3) { /* Zipf over the popularity order */
      pos = s->perm[zipf_draw(t, &s->rng)];
    } else { /* uniform over the allowed range */
      pos = lo_allowed + rng_below(&s->rng, hi_allowed - lo_allowed);
    }
    if (pos >= lo_allowed && pos < hi_allowed && !s->member[pos]) return (int32_t)pos;
  }
  for (int tries = 0; tries < 64; ++tries) {
    int64_t pos = lo_allowed + rng_below(&s->rng, hi_allowed - lo_allowed);
    if (!s->member[pos]) return (int32_t)pos;
  }
  int64_t start = lo_allowed + rng_below(&s->rng, hi_allowed - lo_allowed);
  for (int64_t i = 0; i < hi_allowed - lo_allowed; ++i) {
    int64_t pos = lo_allowed + (start - lo_allowed + i) % (hi_allowed - lo_allowed);
    if (!s->member[pos]) return (int32_t)pos;
  }
  return -1; /* the allowed range is exhausted: leave a pad */
}

/* Redraw `nfresh` of the first `kk` row entries in place (the rest are kept). */
static void redraw_rows(hs_trace_t *t, stream_t *s, int64_t len, int kk, int nfresh, int cls_a,
                        int n_a, int cls_b, int64_t lo_allowed, int64_t hi_allowed) {
  for (int j = 0; j < kk; ++j) s->idx[j] = j;
  for (int i = 0; i < nfresh; ++i) { /* partial Fisher-Yates: idx[0..nfresh) are dropped */
    int j = i + (int)rng_below(&s->rng, kk - i);
    int32_t tmp = s->idx[i]; s->idx[i] = s->idx[j]; s->idx[j] = tmp;
  }
  qsort(s->idx, (size_t)nfresh, sizeof(int32_t), cmp_i32);
  for (int i = 0; i < nfresh; ++i) {
    int32_t old = s->row[s->idx[i]];
    if (old >= 0) s->member[old] = 0;
    s->row[s->idx[i]] = -1;
  }
  for (int i = 0; i < nfresh; ++i) {
    int32_t pos = draw_distinct(t, s, len, i < n_a ? cls_a : cls_b, lo_allowed, hi_allowed);
    s->row[s->idx[i]] = pos;
    if (pos >= 0) s->member[pos] = 1;
  }
}

typedef struct { double score; int32_t page; } scored_t;
static int cmp_scored(const void *a, const void *b) {
  const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
  if (x->score != y->score) return x->score > y->score ? -1 : 1;
  return (x->page > y->page) - (x->page < y->page);
}

/* Advance one decode step.  *appended is set to 1 when every request appends one record at
 * this step (the caller then appends BEFORE resolving with these rows); len_out[N] receives the
 * history length the rows were drawn against.  sel_out is laid out [G][N][k]. */
void hs_trace_step(hs_trace_t *t, int32_t *sel_out, int32_t *appended, int64_t *len_out) {
  const hs_trace_params_t *p = &t->p;
  int N = p->num_requests, G = p->num_streams, k = p->top_k;
  int app = ((t->step + 1) % p->append_every) == 0;
  if (app)
    for (int r = 0; r < N; ++r)
      if (t->len[r] < t->cap[r]) t->len[r]++;
  *appended = app;
  for (int r = 0; r < N; ++r) {
    int64_t len = t->len[r];
    if (len_out) len_out[r] = len;
    for (int g = 0; g < G; ++g) {
      stream_t *s = &t->st[r * G + g];
      int first = !s->started;
      s->started = 1;
      if (p->kind == HS_TRACE_DSA_ZIPF) {
        int nfresh = first ? k : k - p->keep;
        redraw_rows(t, s, len, k, nfresh, 0, nfresh, 0, 0, len);
      } else if (p->kind == HS_TRACE_DSA_MIX) {
        int nfresh = first ? k : k - p->keep;
        redraw_rows(t, s, len, k, nfresh, 1, nfresh / 2, 2, 0, len);
      } else if (p->kind == HS_TRACE_NSA_BLOCKS) {
        int ks = k - 2; /* selected blocks; the last two row entries are the local blocks */
        for (int j = ks; j < k; ++j) { /* drop the old local blocks from the member set */
          if (s->row[j] >= 0) s->member[s->row[j]] = 0;
          s->row[j] = -1;
        }
        int nfresh = first ? ks : ks - p->keep;
        redraw_rows(t, s, len, ks, nfresh, 3, nfresh, 3, 0, p->zipf_support);
        s->row[ks] = (int32_t)(len - 1);
        s->row[ks + 1] = (int32_t)(len - 2);
        s->member[len - 1] = 1; s->member[len - 2] = 1;
      } else { /* HS_TRACE_QUEST_PAGES */
        if (!first) {
          double c = sqrt(1.0 - p->ar_rho * p->ar_rho);
          int64_t old_len = app ? len - 1 : len;
          for (int64_t q = 0; q < old_len; ++q) s->score[q] = p->ar_rho * s->score[q] + c * rng_gauss(&s->rng);
          if (app) s->score[len - 1] = rng_gauss(&s->rng);
        }
        scored_t *sc = (scored_t *)malloc(sizeof(scored_t) * (size_t)len);
        for (int64_t q = 0; q < len; ++q) { sc[q].score = s->score[q]; sc[q].page = (int32_t)q; }
        qsort(sc, (size_t)len, sizeof(scored_t), cmp_scored);
        for (int j = 0; j < k; ++j) s->row[j] = j < len ? sc[j].page : -1;
        free(sc);
      }
      memcpy(sel_out + ((size_t)g * N + r) * k, s->row, sizeof(int32_t) * k);
    }
  }
  t->step++;
}
