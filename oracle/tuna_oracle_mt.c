/*
 * Threaded timing variant of the flat CPU oracle.
 *
 * THIS IS TEST INFRASTRUCTURE, and it is NOT the checker.  The checker is
 * tuna_oracle.c, single-threaded and left as it is.  This file exists only so
 * that a benchmark can say how fast the same rank-by-rank schedule runs when the
 * host's cores share the ranks; a test compares its output, byte for byte and
 * round for round, with the checker's.  Nothing in the CUDA library links,
 * includes or calls it.
 *
 * What it follows: Algorithm 1 with Sec. III-A/B/C of the paper, in the same
 * reading as oracle_tuna_flat (send to the rank at distance +z*r^x; half-open
 * loops; a block is sent in round (x, z) when its x-th digit equals z; a received
 * block is final when no digit above x is non-zero; temporary slots by the map
 * t = o - 1 - dx(r-1) - dz; every rank packs from the state before the round and
 * only then are messages unpacked).  The steps of a round are the same as in the
 * checker; the only difference is who executes them: the "for every rank" loop of
 * the pack step and the one of the unpack step are shared out over plain threads
 * (rank p belongs to thread p mod T), with a barrier between the two steps and
 * one after the round.  A rank only ever writes its own message, its own row of
 * the size table, its own temporary slots and its own region of the receive
 * buffer, so the threads never write the same memory.
 */
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define MT_OK 0
#define MT_EARG -1
#define MT_ENOMEM -2
#define MT_ESCHED -3

#define RS_COLS 6 /* level, x, z, units, bytes sent, bytes received: as in the checker */

static int64_t ipow(int64_t r, int x) {
  int64_t v = 1;
  while (x-- > 0) v *= r;
  return v;
}

static int num_digits(int P, int r) {
  int w = 0;
  int64_t pw = 1;
  while (pw < P) {
    pw *= r;
    w++;
  }
  return w;
}

static int num_rounds(int P, int r) {
  int w = num_digits(P, r), K = 0;
  for (int x = 0; x < w; x++)
    for (int z = 1; z < r; z++)
      if ((int64_t)z * ipow(r, x) < P) K++;
  return K;
}

/* Sec. III-C: slot of offset o in T, or -1 when o is 0 or has a single non-zero digit. */
static int tmap(int P, int r, int o) {
  if (o <= 0 || o >= P) return -1;
  int dx = 0;
  while (ipow(r, dx + 1) <= o) dx++;
  int dz = (int)(o / ipow(r, dx));
  if ((int64_t)dz * ipow(r, dx) == o) return -1;
  return o - 1 - dx * (r - 1) - dz;
}

typedef struct {
  uint8_t *ptr;
  int64_t cap;
} slot_t;

typedef struct {
  int64_t n, bytes;
  int64_t *meta;
  uint8_t *data;
} msg_t;

typedef struct {
  int P, r, elem, B, w, T;
  const int64_t *counts, *sdispls, *rdispls, *sendbase, *recvbase;
  const uint8_t *send;
  uint8_t *recv;
  int64_t *sz;
  slot_t *slots;
  msg_t *msg;
  int *offs;    /* the current round's send set, written by thread 0 between barriers */
  int nsend;
  int64_t *rounds;
  int rounds_cap;
  int64_t *part; /* per thread: units, bytes sent, bytes received of the current round */
  int *status;   /* per thread */
  pthread_barrier_t bar;
  /* start gate: threads wait here until all of them exist (go = 1) or one could
     not be created (go = -1: they leave at once, so no barrier is ever short) */
  pthread_mutex_t gate_lock;
  pthread_cond_t gate;
  int go;
} ctx_t;

typedef struct {
  ctx_t *c;
  int t;
} arg_t;

static void *worker(void *v) {
  arg_t *a = (arg_t *)v;
  ctx_t *c = a->c;
  const int t = a->t, P = c->P, r = c->r, elem = c->elem, B = c->B;
  int k = 0;
  if (t != 0) {
    pthread_mutex_lock(&c->gate_lock);
    while (c->go == 0) pthread_cond_wait(&c->gate, &c->gate_lock);
    const int go = c->go;
    pthread_mutex_unlock(&c->gate_lock);
    if (go < 0) return NULL;
  }
  /* the self block never travels */
  for (int p = t; p < P; p += c->T)
    memcpy(c->recv + (c->recvbase[p] + c->rdispls[(int64_t)p * P + p]) * elem,
           c->send + (c->sendbase[p] + c->sdispls[(int64_t)p * P + p]) * elem,
           (size_t)c->sz[(int64_t)p * P]);
  for (int x = 0; x < c->w; x++) {
    const int64_t rx = ipow(r, x);
    for (int z = 1; z < r; z++) {
      const int64_t dist = z * rx;
      if (dist >= P) continue;
      if (t == 0) { /* the send set of the round: offsets whose x-th digit equals z, ascending */
        int n = 0;
        for (int o = 0; o < P; o++)
          if ((int)((o / rx) % r) == z) c->offs[n++] = o;
        c->nsend = n;
      }
      pthread_barrier_wait(&c->bar);
      const int nsend = c->nsend;
      int64_t units = 0, bsent = 0, brecv = 0;
      /* pack: every rank of this thread, from the state before the round */
      for (int p = t; p < P; p += c->T) {
        msg_t *m = &c->msg[p];
        m->n = nsend;
        m->bytes = 0;
        for (int i = 0; i < nsend; i++) m->bytes += c->sz[(int64_t)p * P + c->offs[i]];
        m->meta = (int64_t *)malloc(sizeof(int64_t) * (size_t)(m->n > 0 ? m->n : 1));
        m->data = (uint8_t *)malloc((size_t)(m->bytes > 0 ? m->bytes : 1));
        if (!m->meta || !m->data) {
          c->status[t] = MT_ENOMEM;
          continue;
        }
        int64_t j = 0, at = 0;
        for (int i = 0; i < nsend; i++) {
          const int o = c->offs[i];
          const int64_t n = c->sz[(int64_t)p * P + o];
          const uint8_t *src;
          if ((o % rx) == 0) {
            src = c->send + (c->sendbase[p] + c->sdispls[(int64_t)p * P + (p + o) % P]) * elem;
          } else {
            const int s = tmap(P, r, o);
            if (s < 0 || s >= B) {
              c->status[t] = MT_ESCHED;
              m->meta[j++] = 0;
              continue;
            }
            src = c->slots[(int64_t)p * B + s].ptr;
          }
          if (n > 0) memcpy(m->data + at, src, (size_t)n);
          m->meta[j++] = n;
          at += n;
        }
        units += m->n;
        bsent += m->bytes;
      }
      pthread_barrier_wait(&c->bar);
      /* unpack: every rank of this thread takes what its partner sent */
      for (int q = t; q < P; q += c->T) {
        const int from = (int)(((q - dist) % P + P) % P);
        const msg_t *m = &c->msg[from];
        if (!m->meta || !m->data) continue;
        int64_t j = 0, at = 0;
        for (int i = 0; i < nsend; i++) {
          const int o = c->offs[i];
          const int64_t n = m->meta[j++];
          c->sz[(int64_t)q * P + o] = n;
          if (o < rx * r) {
            const int src_rank = ((q - o) % P + P) % P;
            memcpy(c->recv + (c->recvbase[q] + c->rdispls[(int64_t)q * P + src_rank]) * elem,
                   m->data + at, (size_t)n);
          } else {
            const int s = tmap(P, r, o);
            if (s < 0 || s >= B) {
              c->status[t] = MT_ESCHED;
            } else {
              slot_t *sl = &c->slots[(int64_t)q * B + s];
              if (n > sl->cap) {
                uint8_t *np_ = (uint8_t *)realloc(sl->ptr, (size_t)n);
                if (!np_) {
                  c->status[t] = MT_ENOMEM;
                  at += n;
                  continue;
                }
                sl->ptr = np_;
                sl->cap = n;
              }
              if (n > 0) memcpy(sl->ptr, m->data + at, (size_t)n);
            }
          }
          at += n;
          brecv += n;
        }
        if (j != m->n || at != m->bytes) c->status[t] = MT_ESCHED;
      }
      c->part[3 * t] = units;
      c->part[3 * t + 1] = bsent;
      c->part[3 * t + 2] = brecv;
      pthread_barrier_wait(&c->bar);
      /* the messages this thread packed have been read by their receivers */
      for (int p = t; p < P; p += c->T) {
        free(c->msg[p].meta);
        free(c->msg[p].data);
        c->msg[p].meta = NULL;
        c->msg[p].data = NULL;
      }
      if (t == 0 && c->rounds && k < c->rounds_cap) {
        int64_t *row = c->rounds + (int64_t)k * RS_COLS;
        row[0] = 0;
        row[1] = x;
        row[2] = z;
        row[3] = row[4] = row[5] = 0;
        for (int u = 0; u < c->T; u++) {
          row[3] += c->part[3 * u];
          row[4] += c->part[3 * u + 1];
          row[5] += c->part[3 * u + 2];
        }
      }
      k++;
    }
  }
  return NULL;
}

/*
 * Algorithm 1 on `threads` plain threads.  Arguments and results as
 * oracle_tuna_flat: counts and displacements in elements of `elem` bytes, `rounds`
 * (may be NULL) receives K rows of RS_COLS values.
 */
int oracle_tuna_flat_mt(int P, int r, int elem, const int64_t *counts, const int64_t *sdispls,
                        const int64_t *rdispls, const int64_t *sendbase, const int64_t *recvbase,
                        const uint8_t *send, uint8_t *recv, int64_t *rounds, int rounds_cap,
                        int threads) {
  if (P < 1 || r < 2 || elem < 1 || threads < 1) return MT_EARG;
  if (threads > P) threads = P;
  ctx_t c;
  memset(&c, 0, sizeof(c));
  c.P = P;
  c.r = r;
  c.elem = elem;
  c.w = num_digits(P, r);
  c.B = P - (num_rounds(P, r) + 1);
  c.T = threads;
  if (c.B < 0) return MT_ESCHED;
  c.counts = counts;
  c.sdispls = sdispls;
  c.rdispls = rdispls;
  c.sendbase = sendbase;
  c.recvbase = recvbase;
  c.send = send;
  c.recv = recv;
  c.rounds = rounds;
  c.rounds_cap = rounds_cap;
  int rc = MT_OK;
  pthread_t *th = (pthread_t *)calloc((size_t)threads, sizeof(pthread_t));
  arg_t *args = (arg_t *)calloc((size_t)threads, sizeof(arg_t));
  c.sz = (int64_t *)malloc(sizeof(int64_t) * (size_t)P * P);
  c.slots = (slot_t *)calloc((size_t)P * (c.B > 0 ? c.B : 1), sizeof(slot_t));
  c.msg = (msg_t *)calloc((size_t)P, sizeof(msg_t));
  c.offs = (int *)malloc(sizeof(int) * (size_t)P);
  c.part = (int64_t *)calloc((size_t)threads * 3, sizeof(int64_t));
  c.status = (int *)calloc((size_t)threads, sizeof(int));
  int started = 0, have_bar = 0;
  if (!th || !args || !c.sz || !c.slots || !c.msg || !c.offs || !c.part || !c.status) {
    rc = MT_ENOMEM;
    goto done;
  }
  for (int p = 0; p < P; p++)
    for (int o = 0; o < P; o++) c.sz[(int64_t)p * P + o] = counts[(int64_t)p * P + (p + o) % P] * elem;
  if (pthread_barrier_init(&c.bar, NULL, (unsigned)threads) != 0) {
    rc = MT_ENOMEM;
    goto done;
  }
  have_bar = 1;
  pthread_mutex_init(&c.gate_lock, NULL);
  pthread_cond_init(&c.gate, NULL);
  for (int t = 1; t < threads; t++) {
    args[t].c = &c;
    args[t].t = t;
    if (pthread_create(&th[t], NULL, worker, &args[t]) != 0) break;
    started = t;
  }
  pthread_mutex_lock(&c.gate_lock);
  c.go = (started == threads - 1) ? 1 : -1;
  pthread_cond_broadcast(&c.gate);
  pthread_mutex_unlock(&c.gate_lock);
  if (c.go < 0) { /* a thread is missing: the others leave at the gate */
    for (int t = 1; t <= started; t++) pthread_join(th[t], NULL);
    rc = MT_ENOMEM;
    goto done;
  }
  args[0].c = &c;
  args[0].t = 0;
  worker(&args[0]);
  for (int t = 1; t < threads; t++) pthread_join(th[t], NULL);
  for (int t = 0; t < threads; t++)
    if (c.status[t] != MT_OK) rc = c.status[t];

done:
  if (have_bar) pthread_barrier_destroy(&c.bar);
  if (c.msg)
    for (int p = 0; p < P; p++) {
      free(c.msg[p].meta);
      free(c.msg[p].data);
    }
  free(c.msg);
  if (c.slots)
    for (int64_t i = 0; i < (int64_t)P * (c.B > 0 ? c.B : 1); i++) free(c.slots[i].ptr);
  free(c.slots);
  free(c.sz);
  free(c.offs);
  free(c.part);
  free(c.status);
  free(th);
  free(args);
  return rc;
}
