/*
 * CPU ORACLE — TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded restatement of HiSparse's per-layer selection resolution,
 * written from the paper's description of the method.  It exists so that tests, the smoke check
 * and the benchmark's CPU-baseline leg have something independent to compare the CUDA path
 * with.  Nothing on the product path may include, link or call this file, and this file shares
 * no code with the CUDA library.
 *
 * The method is an online policy (a particular LRU), so the oracle takes the algorithm's steps
 * one at a time, in the paper's order:
 *   - Sec. 3.2 "KV Hierarchy and Metadata": a B-slot GPU cache per (request, layer), a page
 *     table position -> slot (or host-only), LRU metadata per slot.
 *   - Sec. 3.2 "Replacement policy": LRU per (request, layer); within a step, entries that hit
 *     rank above the newly fetched misses.
 *   - Sec. 3.3 step (3) "Layer decode": find resident selections, fetch the missing records
 *     from the host pool, update page table and LRU, emit device slots aligned with the
 *     selected positions.
 *   - Sec. 3.3 step (4) "Write-through": the newest token's record sits in a reserved slot of
 *     the cache and is written through to the host pool.
 *   - Sec. 3.4 Phase 3: hits to the MRU end, victims assigned to misses, fetched misses just
 *     behind the hits.   Phase 5: page-table update, slots emitted in top-k order.
 *   - Sec. 3.5 "Exact prefetch with shared selections": the anchor records a miss plan (which
 *     host records go to which slots); shared layers replay it and reuse the anchor's table.
 *
 * Readings where the paper is silent (each also listed in the design notes):
 *   - recency is a stamp per slot: 2t+1 for a hit at resolve t, 2t for a record fetched at
 *     resolve t, 0 for a slot never used; victims are taken from slots not hit in this resolve in
 *     ascending (stamp, slot) order; the i-th miss in selection order gets the i-th victim;
 *   - the reserved newest-token slot is slot B, outside the LRU set; selecting the newest
 *     position is a hit on it with no LRU effect;
 *   - -1 is padding (counted neither as hit nor miss); a position outside [0, len) sets the
 *     OUT_OF_RANGE status bit and yields -1; a position repeated in a row sets DUPLICATE, takes
 *     the slot of its first occurrence and is counted neither as hit nor miss.
 *
 * Pins (tests/test_oracle_*.py): the worked example in tests/golden/, an independent ordered-list
 * LRU simulator on tiny random inputs, textbook LRU for k = 1, the B = k "keep only the current
 * top-k" closed form, byte identity with the host history, inverse maps, stamp ordering; for the
 * RANDOM policy's key, the published first outputs of splitmix64 for seed 0 and a key worked out
 * step by step in tests/golden/random_key_worked.txt.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_STATUS_OUT_OF_RANGE 1u
#define ORACLE_STATUS_DUPLICATE 2u
#define ORACLE_FLAG_NO_BYTES 1u /* metadata only: no cache pool, no record copies */

/* Replacement policies.  LRU with hits above misses is the paper's policy (Sec. 3.2); FIFO and RANDOM are the
 * alternatives its cache-locality study replays against the same selection stream (Sec. 4.3, Fig. 6):
 *   FIFO   - a hit does not refresh a slot: stamps record the fetch only, victims are the non-hit slots in
 *            ascending (fetch stamp, slot) order, i-th miss <-> i-th victim;
 *   RANDOM - recency is kept as for LRU but not used for eviction: every non-hit slot gets the key
 *            low32(mix64(mix64(seed ^ (r << 32 | group)) + (t << 32 | slot))), the m smallest (key, slot) are the
 *            victims, and the i-th miss takes the i-th victim in ascending SLOT order. */
#define ORACLE_POLICY_LRU 0
#define ORACLE_POLICY_FIFO 1
#define ORACLE_POLICY_RANDOM 2

typedef struct {
  int N, L, lpg, G, B, k;
  int64_t E;
  uint32_t flags;
  int64_t *cap, *len, *newest;   /* [N] */
  uint8_t **host;                /* [N], caller-owned, layout [L][cap][E] */
  int32_t **slot_pos;            /* [N*G][B]   position held by each slot, -1 = empty */
  uint32_t **last_use;           /* [N*G][B]   recency stamp */
  int32_t **pos2slot;            /* [N*G][cap] page table, -1 = host-only */
  int32_t **first_j;             /* [N*G][cap] scratch for duplicate detection */
  uint32_t *t;                   /* [N*G]      resolves done */
  int32_t **plan_pos, **plan_slot; /* [N*G][k] miss plan of the last anchor resolve */
  int32_t *plan_n;               /* [N*G] */
  int32_t **anchor_out;          /* [N*G][k]   local slots emitted by the last anchor resolve */
  int32_t *anchor_hits, *anchor_misses; /* [N*G] */
  uint8_t **pool;                /* [L] -> [N][B+1][E] */
  uint8_t *replayed;             /* [L] plan replayed into this shared layer since the anchor ran */
  uint32_t status;
  int policy;                    /* ORACLE_POLICY_* */
  uint64_t policy_seed;          /* RANDOM only */
  uint8_t *hit_flag;             /* [B] scratch: slot was hit in the current resolve */
} oracle_t;

static uint8_t *rec_host(oracle_t *o, int r, int l, int64_t p) {
  return o->host[r] + ((int64_t)l * o->cap[r] + p) * o->E;
}
static uint8_t *rec_pool(oracle_t *o, int r, int l, int slot) {
  return o->pool[l] + ((int64_t)r * (o->B + 1) + slot) * o->E;
}

oracle_t *oracle_create(int N, int L, int lpg, int B, int k, int64_t E, const int64_t *cap,
                        const int64_t *init_len, uint8_t *const *host, uint32_t flags) {
  if (N < 1 || L < 1 || lpg < 1 || L % lpg || k < 1 || B < k || E < 1) return NULL;
  oracle_t *o = (oracle_t *)calloc(1, sizeof *o);
  o->N = N; o->L = L; o->lpg = lpg; o->G = L / lpg; o->B = B; o->k = k; o->E = E; o->flags = flags;
  o->cap = (int64_t *)malloc(sizeof(int64_t) * N);
  o->len = (int64_t *)malloc(sizeof(int64_t) * N);
  o->newest = (int64_t *)malloc(sizeof(int64_t) * N);
  o->host = (uint8_t **)malloc(sizeof(uint8_t *) * N);
  for (int r = 0; r < N; ++r) { o->cap[r] = cap[r]; o->len[r] = init_len[r]; o->newest[r] = -1; o->host[r] = host ? host[r] : NULL; }
  int NG = N * o->G;
  o->slot_pos = (int32_t **)malloc(sizeof(void *) * NG);
  o->last_use = (uint32_t **)malloc(sizeof(void *) * NG);
  o->pos2slot = (int32_t **)malloc(sizeof(void *) * NG);
  o->first_j = (int32_t **)malloc(sizeof(void *) * NG);
  o->plan_pos = (int32_t **)malloc(sizeof(void *) * NG);
  o->plan_slot = (int32_t **)malloc(sizeof(void *) * NG);
  o->anchor_out = (int32_t **)malloc(sizeof(void *) * NG);
  o->t = (uint32_t *)calloc(NG, sizeof(uint32_t));
  o->plan_n = (int32_t *)calloc(NG, sizeof(int32_t));
  o->anchor_hits = (int32_t *)calloc(NG, sizeof(int32_t));
  o->anchor_misses = (int32_t *)calloc(NG, sizeof(int32_t));
  for (int r = 0; r < N; ++r)
    for (int g = 0; g < o->G; ++g) {
      int i = r * o->G + g;
      o->slot_pos[i] = (int32_t *)malloc(sizeof(int32_t) * B);
      o->last_use[i] = (uint32_t *)calloc(B, sizeof(uint32_t));
      o->pos2slot[i] = (int32_t *)malloc(sizeof(int32_t) * cap[r]);
      o->first_j[i] = (int32_t *)malloc(sizeof(int32_t) * cap[r]);
      o->plan_pos[i] = (int32_t *)malloc(sizeof(int32_t) * k);
      o->plan_slot[i] = (int32_t *)malloc(sizeof(int32_t) * k);
      o->anchor_out[i] = (int32_t *)malloc(sizeof(int32_t) * k);
      for (int s = 0; s < B; ++s) o->slot_pos[i][s] = -1;
      for (int64_t p = 0; p < cap[r]; ++p) { o->pos2slot[i][p] = -1; o->first_j[i][p] = -1; }
      for (int j = 0; j < k; ++j) o->anchor_out[i][j] = -1;
    }
  o->pool = (uint8_t **)calloc(L, sizeof(void *));
  if (!(flags & ORACLE_FLAG_NO_BYTES))
    for (int l = 0; l < L; ++l) o->pool[l] = (uint8_t *)calloc((size_t)N * (B + 1), (size_t)E);
  o->replayed = (uint8_t *)calloc(L, 1);
  o->hit_flag = (uint8_t *)calloc(B, 1);
  return o;
}

int oracle_set_policy(oracle_t *o, int policy, uint64_t seed) {
  if (policy < ORACLE_POLICY_LRU || policy > ORACLE_POLICY_RANDOM) return -1;
  o->policy = policy;
  o->policy_seed = seed;
  return 0;
}

void oracle_destroy(oracle_t *o) {
  if (!o) return;
  int NG = o->N * o->G;
  for (int i = 0; i < NG; ++i) {
    free(o->slot_pos[i]); free(o->last_use[i]); free(o->pos2slot[i]); free(o->first_j[i]);
    free(o->plan_pos[i]); free(o->plan_slot[i]); free(o->anchor_out[i]);
  }
  for (int l = 0; l < o->L; ++l) free(o->pool[l]);
  free(o->slot_pos); free(o->last_use); free(o->pos2slot); free(o->first_j); free(o->plan_pos);
  free(o->plan_slot); free(o->anchor_out); free(o->t); free(o->plan_n); free(o->anchor_hits);
  free(o->anchor_misses); free(o->pool); free(o->replayed); free(o->cap); free(o->len);
  free(o->newest); free(o->host); free(o->hit_flag); free(o);
}

/* Sec. 3.3 step (4): every request appends one record per layer.  The record goes into the
 * reserved slot B of each layer's cache and is written through to the host history. */
int oracle_append(oracle_t *o, const uint8_t *new_kv /* [N][L][E] */) {
  for (int r = 0; r < o->N; ++r) {
    int64_t p = o->len[r];
    if (p >= o->cap[r]) return -1;
    if (!(o->flags & ORACLE_FLAG_NO_BYTES))
      for (int l = 0; l < o->L; ++l) {
        const uint8_t *src = new_kv + ((int64_t)r * o->L + l) * o->E;
        memcpy(rec_host(o, r, l, p), src, (size_t)o->E);
        memcpy(rec_pool(o, r, l, o->B), src, (size_t)o->E);
      }
    o->newest[r] = p;
    o->len[r] = p + 1;
  }
  return 0;
}

static uint64_t oracle_mix64(uint64_t z) {
  z += 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
static uint32_t random_key(uint64_t seed, int r, int g, uint32_t t, int slot) {
  uint64_t a = oracle_mix64(seed ^ (((uint64_t)(uint32_t)r << 32) | (uint32_t)g));
  return (uint32_t)oracle_mix64(a + (((uint64_t)t << 32) | (uint32_t)slot));
}

/* Accessors for the pins of the two functions above (tests/test_oracle_policies.py): mix64 is the output function
 * of the published splitmix64 generator, whose first outputs for seed 0 are known. */
uint64_t oracle_mix64_value(uint64_t z) { return oracle_mix64(z); }
uint32_t oracle_random_key_value(uint64_t seed, int r, int g, uint32_t t, int slot) { return random_key(seed, r, g, t, slot); }

typedef struct { uint32_t stamp; int32_t slot; } cand_t;
static int cmp_slot(const void *a, const void *b) {
  const cand_t *x = (const cand_t *)a, *y = (const cand_t *)b;
  return (x->slot > y->slot) - (x->slot < y->slot);
}
static int cmp_cand(const void *a, const void *b) {
  const cand_t *x = (const cand_t *)a, *y = (const cand_t *)b;
  if (x->stamp != y->stamp) return x->stamp < y->stamp ? -1 : 1;
  return (x->slot > y->slot) - (x->slot < y->slot);
}

/* Replay the anchor's miss plan into shared layer l (Sec. 3.5): copies only. */
static void replay_plan(oracle_t *o, int l) {
  int g = l / o->lpg;
  if (!(o->flags & ORACLE_FLAG_NO_BYTES))
    for (int r = 0; r < o->N; ++r) {
      int i = r * o->G + g;
      for (int q = 0; q < o->plan_n[i]; ++q)
        memcpy(rec_pool(o, r, l, o->plan_slot[i][q]), rec_host(o, r, l, o->plan_pos[i][q]), (size_t)o->E);
    }
  o->replayed[l] = 1;
}

int oracle_prefetch(oracle_t *o, int layer) {
  if (layer < 0 || layer >= o->L || layer % o->lpg == 0) return -1;
  if (!o->replayed[layer]) replay_plan(o, layer);
  return 0;
}

/* Sec. 3.3 step (3) / Sec. 3.4: resolve one layer for every request.  sel and slot_table are
 * [N][k]; hits and misses are [N]. */
int oracle_resolve(oracle_t *o, int layer, const int32_t *sel, int32_t *slot_table, int32_t *hits,
                   int32_t *misses) {
  if (layer < 0 || layer >= o->L) return -1;
  const int B = o->B, k = o->k, g = layer / o->lpg;
  if (layer % o->lpg != 0) {
    /* shared layer: same selections as its anchor; its cache follows the anchor's slot layout,
     * so the anchor's table is reused once the plan has been replayed into this layer. */
    if (!o->replayed[layer]) replay_plan(o, layer);
    for (int r = 0; r < o->N; ++r) {
      int i = r * o->G + g;
      for (int j = 0; j < k; ++j) {
        int32_t s = o->anchor_out[i][j];
        slot_table[(int64_t)r * k + j] = s < 0 ? -1 : r * (B + 1) + s;
      }
      hits[r] = o->anchor_hits[i];
      misses[r] = o->anchor_misses[i];
    }
    return 0;
  }
  int32_t *out = (int32_t *)malloc(sizeof(int32_t) * k);
  int32_t *dup_of = (int32_t *)malloc(sizeof(int32_t) * k);
  int32_t *miss_j = (int32_t *)malloc(sizeof(int32_t) * k);
  cand_t *cand = (cand_t *)malloc(sizeof(cand_t) * B);
  for (int r = 0; r < o->N; ++r) {
    const int i = r * o->G + g;
    const int32_t *row = sel + (int64_t)r * k;
    int32_t *slot_pos = o->slot_pos[i], *pos2slot = o->pos2slot[i], *first_j = o->first_j[i];
    uint32_t *last_use = o->last_use[i];
    const uint32_t t = ++o->t[i];
    const uint32_t hit_stamp = 2u * t + 1u, miss_stamp = 2u * t;
    int h = 0, m = 0;

    /* pass 1: hits are found and stamped first */
    for (int j = 0; j < k; ++j) {
      int32_t p = row[j];
      out[j] = -1; dup_of[j] = -1;
      if (p == -1) continue;                                   /* padding */
      if (p < 0 || p >= o->len[r]) { o->status |= ORACLE_STATUS_OUT_OF_RANGE; continue; }
      if (first_j[p] >= 0) { o->status |= ORACLE_STATUS_DUPLICATE; dup_of[j] = first_j[p]; continue; }
      first_j[p] = j;
      if (p == o->newest[r]) { out[j] = B; ++h; continue; }   /* reserved newest-token slot */
      int32_t s = pos2slot[p];
      if (s >= 0) { out[j] = s; o->hit_flag[s] = 1; if (o->policy != ORACLE_POLICY_FIFO) last_use[s] = hit_stamp; ++h; }
      else miss_j[m++] = j;
    }

    /* pass 2: eviction candidates = slots not hit in this resolve, ascending (stamp, slot) */
    int nc = 0;
    for (int s = 0; s < B; ++s)
      if (!o->hit_flag[s]) {
        cand[nc].stamp = o->policy == ORACLE_POLICY_RANDOM ? random_key(o->policy_seed, r, g, t, s) : last_use[s];
        cand[nc].slot = s;
        ++nc;
      }
    qsort(cand, (size_t)nc, sizeof(cand_t), cmp_cand);
    if (o->policy == ORACLE_POLICY_RANDOM) qsort(cand, (size_t)(m < nc ? m : nc), sizeof(cand_t), cmp_slot);
    memset(o->hit_flag, 0, (size_t)B);

    /* pass 3: the i-th miss (selection order) takes the i-th candidate */
    for (int q = 0; q < m; ++q) {
      int j = miss_j[q];
      int32_t p = row[j], v = cand[q].slot;
      if (slot_pos[v] >= 0) pos2slot[slot_pos[v]] = -1;        /* evicted record is host-only again */
      slot_pos[v] = p;
      pos2slot[p] = v;
      last_use[v] = miss_stamp;
      if (!(o->flags & ORACLE_FLAG_NO_BYTES))
        memcpy(rec_pool(o, r, layer, v), rec_host(o, r, layer, p), (size_t)o->E);
      o->plan_pos[i][q] = p;
      o->plan_slot[i][q] = v;
      out[j] = v;
    }
    o->plan_n[i] = m;

    /* emit, in selection order */
    for (int j = 0; j < k; ++j) {
      if (dup_of[j] >= 0) out[j] = out[dup_of[j]];
      o->anchor_out[i][j] = out[j];
      slot_table[(int64_t)r * k + j] = out[j] < 0 ? -1 : r * (B + 1) + out[j];
    }
    for (int j = 0; j < k; ++j) {                              /* reset the duplicate scratch */
      int32_t p = row[j];
      if (p >= 0 && p < o->len[r]) first_j[p] = -1;
    }
    hits[r] = h; misses[r] = m;
    o->anchor_hits[i] = h; o->anchor_misses[i] = m;
  }
  for (int l = layer + 1; l < layer + o->lpg; ++l) o->replayed[l] = 0;
  free(out); free(dup_of); free(miss_j); free(cand);
  return 0;
}

/* ---- accessors (state comparison in tests) ---- */
const int32_t *oracle_slot_pos(oracle_t *o, int r, int layer) { return o->slot_pos[r * o->G + layer / o->lpg]; }
const uint32_t *oracle_last_use(oracle_t *o, int r, int layer) { return o->last_use[r * o->G + layer / o->lpg]; }
const int32_t *oracle_pos2slot(oracle_t *o, int r, int layer) { return o->pos2slot[r * o->G + layer / o->lpg]; }
const int32_t *oracle_plan_pos(oracle_t *o, int r, int layer) { return o->plan_pos[r * o->G + layer / o->lpg]; }
const int32_t *oracle_plan_slot(oracle_t *o, int r, int layer) { return o->plan_slot[r * o->G + layer / o->lpg]; }
int32_t oracle_plan_n(oracle_t *o, int r, int layer) { return o->plan_n[r * o->G + layer / o->lpg]; }
const uint8_t *oracle_pool(oracle_t *o, int layer) { return o->pool[layer]; }
int64_t oracle_len(oracle_t *o, int r) { return o->len[r]; }
int64_t oracle_newest(oracle_t *o, int r) { return o->newest[r]; }
uint32_t oracle_steps(oracle_t *o, int r, int layer) { return o->t[r * o->G + layer / o->lpg]; }
uint32_t oracle_status(oracle_t *o) { return o->status; }
void oracle_clear_status(oracle_t *o) { o->status = 0; }

/* Decode KV footprint of Sec. 3.1 "Bounded device footprint": N * L * slots * W_KV * s bytes. */
int64_t oracle_kv_footprint_bytes(int64_t N, int64_t L, int64_t slots, int64_t record_bytes) {
  return N * L * slots * record_bytes;
}
