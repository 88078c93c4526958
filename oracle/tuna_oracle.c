/*
 * CPU oracle for the tunable-radix non-uniform all-to-all (TuNA) and its
 * hierarchical variant.
 *
 * THIS IS TEST INFRASTRUCTURE.  It is a plain, slow, rank-by-rank restatement
 * of the paper's algorithms, used only to check other implementations.  It is
 * not a product path and nothing in the CUDA library links, includes or calls
 * it.
 *
 * What each function follows:
 *   oracle_bruteforce      - the definition of MPI_Alltoallv (Sec. VI-B and the
 *                            Conclusion say the algorithms keep its signature and
 *                            semantics): block j of rank i's send buffer becomes
 *                            block i of rank j's receive buffer.
 *   oracle_num_digits,
 *   oracle_round_list      - Sec. III-A "Tunable Radix": w digits in base r, a
 *                            round is a pair (x, z), 0 <= x < w, 1 <= z < r.
 *   oracle_tmap            - Sec. III-C, the index map t = o - 1 - dx(r-1) - dz
 *                            into the temporary buffer T with B = P-(K+1) slots.
 *   oracle_tuna_flat       - Algorithm 1 with Sec. III-A/B/C.
 *   oracle_tuna_hier       - Sec. IV and Algorithm 3 (coalesced inter-node
 *                            exchange), generalised so that the inter-group
 *                            phase is itself a TuNA of radix rg over
 *                            super-blocks (rg = N gives Algorithm 3's N-1
 *                            rounds of Q blocks each).
 *   oracle_tuna_hier_staggered
 *                          - Sec. IV-B and Algorithm 2: the same local phase, then
 *                            the staggered inter-group exchange, one block per
 *                            step, block_count steps posted per batch.
 *
 *   oracle_rows_alltoallv  - NOT IN THE PAPER: the MPI_Alltoallv definition above with
 *                            a row gather in front of it and a row scatter behind it
 *                            (the token dispatch of a mixture-of-experts layer:
 *                            rows leave in token order and arrive in expert order).
 *                            It is the composition of three textbook definitions
 *                            and is pinned against exactly that composition.
 *
 * Readings taken where the printed text is ambiguous (each pinned by a test):
 *   - direction: a rank sends to the rank at distance +z*r^x (Sec. III-A and the
 *     Fig. 2 narrative: P1 sends to P2 and receives from P0); offsets are
 *     destination minus source.  Algorithm 1's listing prints the mirror image.
 *   - loop bounds are half-open: x < w, 1 <= z < r, offsets < P; rounds whose
 *     distance z*r^x is >= P do not exist (needed for B = 4, 3, 3 at P = 8).
 *   - a block sent in round (x, z) is the one whose x-th digit EQUALS z.
 *   - a received block is final (goes to R) when no digit above x is non-zero,
 *     i.e. offset < r^(x+1); otherwise it goes to T (Sec. III-B/C, Fig. 3).
 *   - dx is the position of the highest non-zero digit (floor of log_r o) and dz
 *     that digit's value; with a ceiling the map is not a bijection for r >= 3.
 *   - every rank packs its message from the state before the round; only then
 *     are messages unpacked (send-receive semantics), so slot reuse in T is safe.
 *   - the self block is copied S -> R and never sent; zero-length blocks keep a
 *     metadata entry and move no bytes.
 *   - blocks inside a message are in ascending offset order.
 *   - Algorithm 2 prints several names for the same quantities; here gi = ii / Q,
 *     gr = ii % Q, the partner groups are (n + gi) mod N for receiving and
 *     (n - gi) mod N for sending (as printed: the mirror image of Algorithm 3's
 *     direction), partner ranks keep the local id q, and block index
 *     group * Q + gr names the block whose original owner has local id gr.
 *
 * All counts and displacements are in elements of elem bytes; rank p's send
 * region starts sendbase[p] elements into `send`, block (p -> d) sits
 * sdispls[p*P+d] elements into that region; recvbase / rdispls[d*P+s] likewise.
 *
 * Parity pins: every function here is pinned by tests (values printed in the
 * paper, closed forms, the brute-force definition); the inter-group phase with
 * radix rg < N has no counterpart in the paper and is pinned only by brute
 * force, byte conservation and its reductions (N = 1, Q = 1, rg = N).
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_EARG -1
#define ORACLE_ENOMEM -2
#define ORACLE_ESCHED -3 /* an internal invariant of the schedule failed */

/* one row of the per-round statistics table */
#define RS_LEVEL 0 /* 0 = flat or local, 1 = global */
#define RS_X 1
#define RS_Z 2
#define RS_UNITS 3 /* blocks (level 0) or super-blocks (level 1) sent, all ranks */
#define RS_BYTES_SENT 4
#define RS_BYTES_RECV 5
#define RS_COLS 6

/* one row of the optional trace of a single rank */
#define TR_ROUND 0
#define TR_KIND 1    /* 0 = sent by the traced rank, 1 = received by it */
#define TR_PARTNER 2 /* rank sent to / received from */
#define TR_OFFSET 3
#define TR_ORIGIN 4  /* rank that owns the block originally */
#define TR_DEST 5    /* rank the block is finally for */
#define TR_BYTES 6
#define TR_PLACE 7   /* sent: 0 = read from S, 2 = read from T; received: 1 = R, 2 = T */
#define TR_COLS 8

static int64_t ipow(int64_t r, int x) {
  int64_t v = 1;
  while (x-- > 0) v *= r;
  return v;
}

static int digit_of(int64_t o, int r, int x) { return (int)((o / ipow(r, x)) % r); }

/* The send set of round (x, z): offsets below `count` whose x-th base-r digit
   equals z, ascending (Sec. III-A).  Returns how many. */
static int send_offsets(int count, int r, int x, int z, int *out) {
  int n = 0;
  for (int o = 0; o < count; o++)
    if (digit_of(o, r, x) == z) out[n++] = o;
  return n;
}

/* Sec. III-A: number of base-r digits needed for P block indices. */
int oracle_num_digits(int P, int r) {
  int w = 0;
  int64_t pw = 1;
  if (P < 1 || r < 2) return -1;
  while (pw < P) {
    pw *= r;
    w++;
  }
  return w;
}

/* Sec. III-A: the rounds (x, z) in execution order; returns K. */
int oracle_round_list(int P, int r, int *xs, int *zs, int cap) {
  int w = oracle_num_digits(P, r), K = 0;
  if (w < 0) return -1;
  for (int x = 0; x < w; x++)
    for (int z = 1; z < r; z++) {
      if ((int64_t)z * ipow(r, x) >= P) continue;
      if (xs && zs && K < cap) {
        xs[K] = x;
        zs[K] = z;
      }
      K++;
    }
  return K;
}

/* Sec. III-C: slot of offset o in T, or -1 when o is 0 (self) or direct. */
int oracle_tmap(int P, int r, int o) {
  if (o <= 0 || o >= P) return -1;
  int dx = 0;
  while (ipow(r, dx + 1) <= o) dx++;
  int dz = (int)(o / ipow(r, dx));
  if ((int64_t)dz * ipow(r, dx) == o) return -1; /* a single non-zero digit */
  return o - 1 - dx * (r - 1) - dz;
}

/* Definition of the exchange. */
int oracle_bruteforce(int P, int elem, const int64_t *counts, const int64_t *sdispls,
                      const int64_t *rdispls, const int64_t *sendbase,
                      const int64_t *recvbase, const uint8_t *send, uint8_t *recv) {
  if (P < 1 || elem < 1) return ORACLE_EARG;
  for (int s = 0; s < P; s++)
    for (int d = 0; d < P; d++) {
      int64_t n = counts[(int64_t)s * P + d] * elem;
      const uint8_t *src = send + (sendbase[s] + sdispls[(int64_t)s * P + d]) * elem;
      uint8_t *dst = recv + (recvbase[d] + rdispls[(int64_t)d * P + s]) * elem;
      memcpy(dst, src, (size_t)n);
    }
  return ORACLE_OK;
}

/* Segmented exclusive prefix sum, the textbook running sum: nseg segments of
   seglen values; each value is first rounded up to a multiple of `align`
   (align = 1: no rounding).  out[s][i] = sum of the rounded values before i in
   segment s; totals[s] (may be NULL) = the segment's sum.  These sums are what
   turns a rank's list of block sizes into displacements (Sec. III-B/C). */
int oracle_segmented_exclusive_scan(const int64_t *val, int64_t nseg, int64_t seglen,
                                    int64_t align, int64_t *out, int64_t *totals) {
  if (nseg < 0 || seglen < 0 || align < 1) return ORACLE_EARG;
  for (int64_t s = 0; s < nseg; s++) {
    int64_t run = 0;
    for (int64_t i = 0; i < seglen; i++) {
      int64_t v = val[s * seglen + i];
      v = (v + align - 1) / align * align;
      out[s * seglen + i] = run;
      run += v;
    }
    if (totals) totals[s] = run;
  }
  return ORACLE_OK;
}

/* ---- small helpers shared by the two schedules ---- */

typedef struct {
  uint8_t *ptr;
  int64_t cap;
} slot_t;

static int slot_put(slot_t *s, const uint8_t *src, int64_t n) {
  if (n > s->cap) {
    uint8_t *p = (uint8_t *)realloc(s->ptr, (size_t)n);
    if (!p) return ORACLE_ENOMEM;
    s->ptr = p;
    s->cap = n;
  }
  if (n > 0) memcpy(s->ptr, src, (size_t)n);
  return ORACLE_OK;
}

typedef struct {
  int64_t n;       /* blocks in the message */
  int64_t *meta;   /* metadata message: their sizes in bytes */
  uint8_t *data;   /* data message: the blocks back to back */
  int64_t bytes;
} msg_t;

static void msg_free(msg_t *m) {
  free(m->meta);
  free(m->data);
  m->meta = NULL;
  m->data = NULL;
}

static void trace_row(int64_t *trace, int64_t cap, int64_t *rows, int64_t round, int64_t kind,
                      int64_t partner, int64_t off, int64_t origin, int64_t dest, int64_t bytes,
                      int64_t place) {
  if (!trace || !rows) return;
  if (*rows < cap) {
    int64_t *t = trace + *rows * TR_COLS;
    t[TR_ROUND] = round;
    t[TR_KIND] = kind;
    t[TR_PARTNER] = partner;
    t[TR_OFFSET] = off;
    t[TR_ORIGIN] = origin;
    t[TR_DEST] = dest;
    t[TR_BYTES] = bytes;
    t[TR_PLACE] = place;
  }
  (*rows)++;
}

/*
 * Algorithm 1.  `rounds` (may be NULL) receives K rows of RS_COLS values;
 * `trace` (may be NULL) receives what rank `trace_rank` sent and received.
 * `tslots_out` (may be NULL) receives B, the number of T slots per rank.
 * `sz_phases` (may be NULL, w*P*P values) receives, after all rounds of digit
 * position x, the metadata every rank holds: sz_phases[x][p][o] = bytes of the
 * block rank p holds for offset o (Sec. III-B: sizes travel ahead of the data).
 */
int oracle_tuna_flat(int P, int r, int elem, const int64_t *counts, const int64_t *sdispls,
                     const int64_t *rdispls, const int64_t *sendbase, const int64_t *recvbase,
                     const uint8_t *send, uint8_t *recv, int64_t *rounds, int rounds_cap,
                     int *K_out, int *tslots_out, int trace_rank, int64_t *trace,
                     int64_t trace_cap, int64_t *trace_rows, int64_t *sz_phases) {
  if (P < 1 || r < 2 || elem < 1) return ORACLE_EARG;
  int rc = ORACLE_OK;
  int w = oracle_num_digits(P, r);
  int K = oracle_round_list(P, r, NULL, NULL, 0);
  int B = P - (K + 1); /* Sec. III-C */
  if (B < 0) return ORACLE_ESCHED;
  if (K_out) *K_out = K;
  if (tslots_out) *tslots_out = B;
  if (trace_rows) *trace_rows = 0;

  /* sz[p][o]: size in bytes of the block rank p currently holds for offset o.
     Naming blocks by offset is the index-only "rotation": no data moves. */
  int64_t *sz = (int64_t *)malloc(sizeof(int64_t) * (size_t)P * P);
  slot_t *T = (slot_t *)calloc((size_t)P * (B > 0 ? B : 1), sizeof(slot_t));
  msg_t *msg = (msg_t *)calloc((size_t)P, sizeof(msg_t));
  int *offs = (int *)malloc(sizeof(int) * (size_t)P);
  if (!sz || !T || !msg || !offs) {
    rc = ORACLE_ENOMEM;
    goto done;
  }
  for (int p = 0; p < P; p++)
    for (int o = 0; o < P; o++) sz[(int64_t)p * P + o] = counts[(int64_t)p * P + (p + o) % P] * elem;

  /* the self block never travels */
  for (int p = 0; p < P; p++)
    memcpy(recv + (recvbase[p] + rdispls[(int64_t)p * P + p]) * elem,
           send + (sendbase[p] + sdispls[(int64_t)p * P + p]) * elem, (size_t)sz[(int64_t)p * P]);

  int k = 0;
  for (int x = 0; x < w; x++) {
    int64_t rx = ipow(r, x);
    for (int z = 1; z < r; z++) {
      int64_t dist = z * rx;
      if (dist >= P) continue;
      int64_t units = 0, bsent = 0, brecv = 0;
      const int nsend = send_offsets(P, r, x, z, offs);

      /* every rank packs its metadata and data messages from the pre-round state */
      for (int p = 0; p < P; p++) {
        msg_t *m = &msg[p];
        int to = (int)((p + dist) % P);
        m->n = nsend;
        m->bytes = 0;
        for (int a = 0; a < nsend; a++) m->bytes += sz[(int64_t)p * P + offs[a]];
        m->meta = (int64_t *)malloc(sizeof(int64_t) * (size_t)(m->n > 0 ? m->n : 1));
        m->data = (uint8_t *)malloc((size_t)(m->bytes > 0 ? m->bytes : 1));
        if (!m->meta || !m->data) {
          rc = ORACLE_ENOMEM;
          goto done;
        }
        int64_t j = 0, at = 0;
        for (int a = 0; a < nsend; a++) {
          const int o = offs[a];
          int64_t n = sz[(int64_t)p * P + o];
          int from_T = (o % rx) != 0; /* it has already travelled: it sits in T */
          const uint8_t *src;
          if (!from_T) {
            src = send + (sendbase[p] + sdispls[(int64_t)p * P + (p + o) % P]) * elem;
          } else {
            int t = oracle_tmap(P, r, o);
            if (t < 0 || t >= B) {
              rc = ORACLE_ESCHED;
              goto done;
            }
            src = T[(int64_t)p * B + t].ptr;
          }
          if (n > 0) memcpy(m->data + at, src, (size_t)n);
          m->meta[j++] = n;
          at += n;
          if (p == trace_rank) {
            int origin = (int)(((p - (o % rx)) % P + P) % P);
            trace_row(trace, trace_cap, trace_rows, k, 0, to, o, origin, (origin + o) % P, n,
                      from_T ? 2 : 0);
          }
        }
        units += m->n;
        bsent += m->bytes;
      }

      /* every rank unpacks what its partner sent */
      for (int q = 0; q < P; q++) {
        int from = (int)(((q - dist) % P + P) % P);
        msg_t *m = &msg[from];
        int64_t j = 0, at = 0;
        for (int a = 0; a < nsend; a++) {
          const int o = offs[a];
          int64_t n = m->meta[j++];
          sz[(int64_t)q * P + o] = n; /* phase 1: the metadata */
          int final = o < rx * r;     /* no non-zero digit above x */
          if (final) {
            int src_rank = ((q - o) % P + P) % P;
            memcpy(recv + (recvbase[q] + rdispls[(int64_t)q * P + src_rank]) * elem, m->data + at,
                   (size_t)n);
          } else {
            int t = oracle_tmap(P, r, o);
            if (t < 0 || t >= B) {
              rc = ORACLE_ESCHED;
              goto done;
            }
            rc = slot_put(&T[(int64_t)q * B + t], m->data + at, n);
            if (rc) goto done;
          }
          at += n;
          brecv += n;
          if (q == trace_rank) {
            int origin = (int)(((q - (o % (rx * r))) % P + P) % P);
            trace_row(trace, trace_cap, trace_rows, k, 1, from, o, origin, (origin + o) % P, n,
                      final ? 1 : 2);
          }
        }
        if (j != m->n || at != m->bytes) {
          rc = ORACLE_ESCHED;
          goto done;
        }
      }
      for (int p = 0; p < P; p++) msg_free(&msg[p]);

      if (rounds && k < rounds_cap) {
        int64_t *row = rounds + (int64_t)k * RS_COLS;
        row[RS_LEVEL] = 0;
        row[RS_X] = x;
        row[RS_Z] = z;
        row[RS_UNITS] = units;
        row[RS_BYTES_SENT] = bsent;
        row[RS_BYTES_RECV] = brecv;
      }
      k++;
    }
    if (sz_phases) memcpy(sz_phases + (int64_t)x * P * P, sz, sizeof(int64_t) * (size_t)P * P);
  }
  if (k != K) rc = ORACLE_ESCHED;

done:
  if (msg)
    for (int p = 0; p < P; p++) msg_free(&msg[p]);
  free(msg);
  if (T)
    for (int64_t i = 0; i < (int64_t)P * (B > 0 ? B : 1); i++) free(T[i].ptr);
  free(T);
  free(sz);
  free(offs);
  return rc;
}

/*
 * Sec. IV / Algorithm 3.  P = Q*N ranks, rank p = n*Q + q (consecutive ranks
 * form a group).  Local phase: N concurrent Q x Q TuNA exchanges of radix rl
 * inside every group (the implicit strategy); own-group blocks end in R, the
 * others are kept, compacted into one super-block per destination group, and
 * then exchanged between the ranks that share local id q by a TuNA of radix rg
 * over the N groups whose unit is the super-block.
 *
 * `recv_after_local` (may be NULL) receives a copy of the receive buffer as it
 * stands after the local phase.  K_out[0] = local rounds, K_out[1] = global.
 * Three more optional outputs copy out the metadata the ranks hold (Sec. III-B:
 * sizes travel ahead of the data), without touching it:
 *   sz_local     wl*P*P values: after all rounds of local digit position x,
 *                sz_local[x][p][i*Q + jo] = bytes of the block rank p = (n, q) holds
 *                for rank (i, (q + jo) % Q);
 *   usz_compact  P*N*Q values: after the compaction (Sec. IV-B),
 *                usz_compact[p][io][q'] = bytes of the part that came from rank
 *                (n, q') in the super-block rank p holds for group (n + io) % N;
 *   usz_global   wg*P*N*Q values: the same table after all rounds of global digit
 *                position x.
 */
static int hier_impl(int Q, int N, int rl, int rg, int block_count, int elem,
                     const int64_t *counts, const int64_t *sdispls, const int64_t *rdispls,
                     const int64_t *sendbase, const int64_t *recvbase, const uint8_t *send,
                     uint8_t *recv, int64_t recv_bytes, uint8_t *recv_after_local,
                     int64_t *rounds, int rounds_cap, int *K_out, int *batches_out,
                     int64_t *sz_local, int64_t *usz_compact, int64_t *usz_global) {
  if (Q < 1 || N < 1 || rl < 2 || rg < 2 || elem < 1 || block_count < 0) return ORACLE_EARG;
  const int P = Q * N;
  int rc = ORACLE_OK;
  const int wl = oracle_num_digits(Q, rl), wg = oracle_num_digits(N, rg);
  const int Kl = oracle_round_list(Q, rl, NULL, NULL, 0);
  const int Kg = block_count > 0 ? Q * (N - 1) : oracle_round_list(N, rg, NULL, NULL, 0);
  const int Bg = block_count > 0 ? 0 : N - (Kg + 1);
  if (Bg < 0) return ORACLE_ESCHED;
  if (K_out) {
    K_out[0] = Kl;
    K_out[1] = Kg;
  }
  slot_t *box = NULL;     /* staggered exchange: blocks in flight within a batch */
  int64_t *boxlen = NULL; /* and their sizes */

  /* local phase state: slot (i, jo) of rank (n, q) names the block for rank
     (i, (q + jo) % Q); sz holds its current size, L its bytes once it has moved */
  int64_t *sz = (int64_t *)malloc(sizeof(int64_t) * (size_t)P * P);
  slot_t *L = (slot_t *)calloc((size_t)P * P, sizeof(slot_t));
  msg_t *msg = (msg_t *)calloc((size_t)P, sizeof(msg_t));
  /* global phase state */
  slot_t *U = (slot_t *)calloc((size_t)P * N, sizeof(slot_t));  /* super-blocks by dest group */
  int64_t *usz = (int64_t *)calloc((size_t)P * N * Q, sizeof(int64_t)); /* [p][io][q'] */
  slot_t *TG = (slot_t *)calloc((size_t)P * (Bg > 0 ? Bg : 1), sizeof(slot_t));
  int *offs = (int *)malloc(sizeof(int) * (size_t)(Q > N ? Q : N));
  if (!sz || !L || !msg || !U || !usz || !TG || !offs) {
    rc = ORACLE_ENOMEM;
    goto done;
  }
  for (int p = 0; p < P; p++) {
    int n = p / Q, q = p % Q;
    (void)n;
    for (int i = 0; i < N; i++)
      for (int jo = 0; jo < Q; jo++)
        sz[(int64_t)p * P + i * Q + jo] = counts[(int64_t)p * P + i * Q + (q + jo) % Q] * elem;
  }
  /* the self block */
  for (int p = 0; p < P; p++)
    memcpy(recv + (recvbase[p] + rdispls[(int64_t)p * P + p]) * elem,
           send + (sendbase[p] + sdispls[(int64_t)p * P + p]) * elem,
           (size_t)(counts[(int64_t)p * P + p] * elem));

  int k = 0;
  for (int x = 0; x < wl; x++) {
    int64_t rx = ipow(rl, x);
    for (int z = 1; z < rl; z++) {
      int64_t dist = z * rx;
      if (dist >= Q) continue;
      int64_t units = 0, bsent = 0, brecv = 0;
      const int nsend = send_offsets(Q, rl, x, z, offs);
      for (int p = 0; p < P; p++) {
        int n = p / Q, q = p % Q;
        msg_t *m = &msg[p];
        m->n = (int64_t)N * nsend;
        m->bytes = 0;
        for (int i = 0; i < N; i++)
          for (int a = 0; a < nsend; a++) m->bytes += sz[(int64_t)p * P + i * Q + offs[a]];
        m->meta = (int64_t *)malloc(sizeof(int64_t) * (size_t)(m->n > 0 ? m->n : 1));
        m->data = (uint8_t *)malloc((size_t)(m->bytes > 0 ? m->bytes : 1));
        if (!m->meta || !m->data) {
          rc = ORACLE_ENOMEM;
          goto done;
        }
        int64_t j = 0, at = 0;
        for (int i = 0; i < N; i++)
          for (int a = 0; a < nsend; a++) {
            const int jo = offs[a];
            int64_t nb = sz[(int64_t)p * P + i * Q + jo];
            const uint8_t *src;
            if (jo % rx == 0) /* still where its owner put it */
              src = send + (sendbase[p] + sdispls[(int64_t)p * P + i * Q + (q + jo) % Q]) * elem;
            else
              src = L[(int64_t)p * P + i * Q + jo].ptr;
            if (nb > 0) memcpy(m->data + at, src, (size_t)nb);
            m->meta[j++] = nb;
            at += nb;
          }
        (void)n;
        units += m->n;
        bsent += m->bytes;
      }
      for (int p = 0; p < P; p++) {
        int n = p / Q, q = p % Q;
        int from = n * Q + (int)(((q - dist) % Q + Q) % Q);
        msg_t *m = &msg[from];
        int64_t j = 0, at = 0;
        for (int i = 0; i < N; i++)
          for (int a = 0; a < nsend; a++) {
            const int jo = offs[a];
            int64_t nb = m->meta[j++];
            sz[(int64_t)p * P + i * Q + jo] = nb;
            int local_final = jo < rx * rl;
            if (local_final && i == n) {
              int src_rank = n * Q + ((q - jo) % Q + Q) % Q;
              memcpy(recv + (recvbase[p] + rdispls[(int64_t)p * P + src_rank]) * elem,
                     m->data + at, (size_t)nb);
            } else {
              rc = slot_put(&L[(int64_t)p * P + i * Q + jo], m->data + at, nb);
              if (rc) goto done;
            }
            at += nb;
            brecv += nb;
          }
        if (j != m->n || at != m->bytes) {
          rc = ORACLE_ESCHED;
          goto done;
        }
      }
      for (int p = 0; p < P; p++) msg_free(&msg[p]);
      if (rounds && k < rounds_cap) {
        int64_t *row = rounds + (int64_t)k * RS_COLS;
        row[RS_LEVEL] = 0;
        row[RS_X] = x;
        row[RS_Z] = z;
        row[RS_UNITS] = units;
        row[RS_BYTES_SENT] = bsent;
        row[RS_BYTES_RECV] = brecv;
      }
      k++;
    }
    if (sz_local) memcpy(sz_local + (int64_t)x * P * P, sz, sizeof(int64_t) * (size_t)P * P);
  }
  if (k != Kl) {
    rc = ORACLE_ESCHED;
    goto done;
  }
  if (recv_after_local) memcpy(recv_after_local, recv, (size_t)recv_bytes);

  if (block_count > 0) {
    /* Algorithm 2, the staggered inter-group exchange.  A step index ii runs
       over [0, P) in batches of block_count; step ii stands for the pair
       gi = ii / Q (group distance) and gr = ii % Q (local id of the block's
       original owner).  In step (gi, gr) with gi >= 1, rank (n, q) sends the
       single block that came from rank (n, gr) and is meant for rank
       ((n - gi) mod N, q) to that rank, and receives from rank
       ((n + gi) mod N, q) the block that came from ((n + gi) mod N, gr).  Steps
       with gi = 0 name the rank's own group and do nothing.  The receiver knows
       the size from its receive counts, so no metadata travels and nothing is
       compacted.  Within a batch every receive and send is posted before any
       completes: all ranks hand their blocks over, then all take delivery. */
    int batches = 0;
    box = (slot_t *)calloc((size_t)P * block_count, sizeof(slot_t));
    boxlen = (int64_t *)calloc((size_t)P * block_count, sizeof(int64_t));
    if (!box || !boxlen) {
      rc = ORACLE_ENOMEM;
      goto done;
    }
    for (int r0 = 0; r0 < Kg && rounds && Kl + r0 < rounds_cap; r0++) {
      int64_t *row = rounds + (int64_t)(Kl + r0) * RS_COLS;
      row[RS_LEVEL] = 1;
      row[RS_X] = 1 + r0 / Q;
      row[RS_Z] = r0 % Q;
      row[RS_UNITS] = 0;
      row[RS_BYTES_SENT] = 0;
      row[RS_BYTES_RECV] = 0;
    }
    for (int ii = 0; ii < P; ii += block_count) {
      int active = 0;
      for (int p = 0; p < P; p++) {
        int n = p / Q, q = p % Q;
        for (int i = 0; i < block_count && ii + i < P; i++) {
          int gi = (ii + i) / Q, gr = (ii + i) % Q;
          int ndst = ((n - gi) % N + N) % N;
          if (ndst == n) continue;
          active = 1;
          int jo = ((q - gr) % Q + Q) % Q;
          int64_t nb = sz[(int64_t)p * P + ndst * Q + jo];
          const uint8_t *src = (jo == 0)
                                   ? send + (sendbase[p] + sdispls[(int64_t)p * P + ndst * Q + q]) * elem
                                   : L[(int64_t)p * P + ndst * Q + jo].ptr;
          rc = slot_put(&box[(int64_t)p * block_count + i], src, nb);
          if (rc) goto done;
          boxlen[(int64_t)p * block_count + i] = nb;
          if (rounds && Kl + (gi - 1) * Q + gr < rounds_cap) {
            int64_t *row = rounds + (int64_t)(Kl + (gi - 1) * Q + gr) * RS_COLS;
            row[RS_UNITS] += 1;
            row[RS_BYTES_SENT] += nb;
          }
        }
      }
      for (int p = 0; p < P; p++) {
        int n = p / Q, q = p % Q;
        for (int i = 0; i < block_count && ii + i < P; i++) {
          int gi = (ii + i) / Q, gr = (ii + i) % Q;
          int nsrc = (n + gi) % N;
          if (nsrc == n) continue;
          const slot_t *b = &box[(int64_t)(nsrc * Q + q) * block_count + i];
          int64_t want = counts[(int64_t)(nsrc * Q + gr) * P + p] * elem;
          if (boxlen[(int64_t)(nsrc * Q + q) * block_count + i] != want) {
            rc = ORACLE_ESCHED;
            goto done;
          }
          if (want > 0)
            memcpy(recv + (recvbase[p] + rdispls[(int64_t)p * P + nsrc * Q + gr]) * elem, b->ptr,
                   (size_t)want);
          if (rounds && Kl + (gi - 1) * Q + gr < rounds_cap)
            rounds[(int64_t)(Kl + (gi - 1) * Q + gr) * RS_COLS + RS_BYTES_RECV] += want;
        }
      }
      batches += active;
    }
    if (batches_out) *batches_out = batches;
    goto done;
  }

  /* compaction: rank (n, q) gathers, for every other group i, the Q blocks
     (n, q') -> (i, q) in ascending q' into one contiguous super-block */
  for (int p = 0; p < P; p++) {
    int n = p / Q, q = p % Q;
    for (int i = 0; i < N; i++) {
      if (i == n) continue;
      int io = ((i - n) % N + N) % N;
      int64_t tot = 0;
      for (int qs = 0; qs < Q; qs++) {
        int jo = ((q - qs) % Q + Q) % Q;
        int64_t nb = sz[(int64_t)p * P + i * Q + jo];
        usz[((int64_t)p * N + io) * Q + qs] = nb;
        tot += nb;
      }
      slot_t *u = &U[(int64_t)p * N + io];
      u->ptr = (uint8_t *)malloc((size_t)(tot > 0 ? tot : 1));
      if (!u->ptr) {
        rc = ORACLE_ENOMEM;
        goto done;
      }
      u->cap = tot;
      int64_t at = 0;
      for (int qs = 0; qs < Q; qs++) {
        int jo = ((q - qs) % Q + Q) % Q;
        int64_t nb = usz[((int64_t)p * N + io) * Q + qs];
        const uint8_t *src = (jo == 0)
                                 ? send + (sendbase[p] + sdispls[(int64_t)p * P + i * Q + q]) * elem
                                 : L[(int64_t)p * P + i * Q + jo].ptr;
        if (nb > 0) memcpy(u->ptr + at, src, (size_t)nb);
        at += nb;
      }
    }
  }

  if (usz_compact) memcpy(usz_compact, usz, sizeof(int64_t) * (size_t)P * N * Q);

  /* global phase: Algorithm 1 over the N ranks with the same q; the unit is a
     super-block, its metadata the Q sizes of its parts */
  for (int x = 0; x < wg; x++) {
    int64_t rx = ipow(rg, x);
    for (int z = 1; z < rg; z++) {
      int64_t dist = z * rx;
      if (dist >= N) continue;
      int64_t units = 0, bsent = 0, brecv = 0;
      const int nsend = send_offsets(N, rg, x, z, offs);
      for (int p = 0; p < P; p++) {
        msg_t *m = &msg[p];
        m->n = nsend;
        m->bytes = 0;
        for (int a = 0; a < nsend; a++)
          for (int qs = 0; qs < Q; qs++) m->bytes += usz[((int64_t)p * N + offs[a]) * Q + qs];
        m->meta = (int64_t *)malloc(sizeof(int64_t) * (size_t)(m->n > 0 ? m->n * Q : 1));
        m->data = (uint8_t *)malloc((size_t)(m->bytes > 0 ? m->bytes : 1));
        if (!m->meta || !m->data) {
          rc = ORACLE_ENOMEM;
          goto done;
        }
        int64_t j = 0, at = 0;
        for (int a = 0; a < nsend; a++) {
          const int io = offs[a];
          int64_t tot = 0;
          for (int qs = 0; qs < Q; qs++) {
            int64_t nb = usz[((int64_t)p * N + io) * Q + qs];
            m->meta[j * Q + qs] = nb;
            tot += nb;
          }
          const uint8_t *src;
          if (io % rx == 0) {
            src = U[(int64_t)p * N + io].ptr;
          } else {
            int t = oracle_tmap(N, rg, io);
            if (t < 0 || t >= Bg) {
              rc = ORACLE_ESCHED;
              goto done;
            }
            src = TG[(int64_t)p * Bg + t].ptr;
          }
          if (tot > 0) memcpy(m->data + at, src, (size_t)tot);
          at += tot;
          j++;
        }
        units += m->n;
        bsent += m->bytes;
      }
      for (int p = 0; p < P; p++) {
        int n = p / Q, q = p % Q;
        int from = (int)(((n - dist) % N + N) % N) * Q + q;
        msg_t *m = &msg[from];
        int64_t j = 0, at = 0;
        for (int a = 0; a < nsend; a++) {
          const int io = offs[a];
          int64_t tot = 0;
          for (int qs = 0; qs < Q; qs++) {
            int64_t nb = m->meta[j * Q + qs];
            usz[((int64_t)p * N + io) * Q + qs] = nb;
            tot += nb;
          }
          if (io < rx * rg) { /* final: split the super-block into R */
            int src_group = ((n - io) % N + N) % N;
            int64_t a = at;
            for (int qs = 0; qs < Q; qs++) {
              int64_t nb = m->meta[j * Q + qs];
              memcpy(recv + (recvbase[p] + rdispls[(int64_t)p * P + src_group * Q + qs]) * elem,
                     m->data + a, (size_t)nb);
              a += nb;
            }
          } else {
            int t = oracle_tmap(N, rg, io);
            if (t < 0 || t >= Bg) {
              rc = ORACLE_ESCHED;
              goto done;
            }
            rc = slot_put(&TG[(int64_t)p * Bg + t], m->data + at, tot);
            if (rc) goto done;
          }
          at += tot;
          brecv += tot;
          j++;
        }
        if (j != m->n || at != m->bytes) {
          rc = ORACLE_ESCHED;
          goto done;
        }
      }
      for (int p = 0; p < P; p++) msg_free(&msg[p]);
      if (rounds && k < rounds_cap) {
        int64_t *row = rounds + (int64_t)k * RS_COLS;
        row[RS_LEVEL] = 1;
        row[RS_X] = x;
        row[RS_Z] = z;
        row[RS_UNITS] = units;
        row[RS_BYTES_SENT] = bsent;
        row[RS_BYTES_RECV] = brecv;
      }
      k++;
    }
    if (usz_global)
      memcpy(usz_global + (int64_t)x * P * N * Q, usz, sizeof(int64_t) * (size_t)P * N * Q);
  }
  if (k != Kl + Kg) rc = ORACLE_ESCHED;

done:
  free(offs);
  if (msg)
    for (int p = 0; p < P; p++) msg_free(&msg[p]);
  free(msg);
  if (box)
    for (int64_t i = 0; i < (int64_t)P * block_count; i++) free(box[i].ptr);
  free(box);
  free(boxlen);
  if (L)
    for (int64_t i = 0; i < (int64_t)P * P; i++) free(L[i].ptr);
  free(L);
  if (U)
    for (int64_t i = 0; i < (int64_t)P * N; i++) free(U[i].ptr);
  free(U);
  if (TG)
    for (int64_t i = 0; i < (int64_t)P * (Bg > 0 ? Bg : 1); i++) free(TG[i].ptr);
  free(TG);
  free(usz);
  free(sz);
  return rc;
}

int oracle_tuna_hier(int Q, int N, int rl, int rg, int elem, const int64_t *counts,
                     const int64_t *sdispls, const int64_t *rdispls, const int64_t *sendbase,
                     const int64_t *recvbase, const uint8_t *send, uint8_t *recv,
                     int64_t recv_bytes, uint8_t *recv_after_local, int64_t *rounds,
                     int rounds_cap, int *K_out) {
  return hier_impl(Q, N, rl, rg, 0, elem, counts, sdispls, rdispls, sendbase, recvbase, send, recv,
                   recv_bytes, recv_after_local, rounds, rounds_cap, K_out, NULL, NULL, NULL, NULL);
}

/* oracle_tuna_hier with the metadata tables of hier_impl copied out as well. */
int oracle_tuna_hier_tables(int Q, int N, int rl, int rg, int elem, const int64_t *counts,
                            const int64_t *sdispls, const int64_t *rdispls,
                            const int64_t *sendbase, const int64_t *recvbase,
                            const uint8_t *send, uint8_t *recv, int64_t recv_bytes,
                            uint8_t *recv_after_local, int64_t *sz_local, int64_t *usz_compact,
                            int64_t *usz_global) {
  return hier_impl(Q, N, rl, rg, 0, elem, counts, sdispls, rdispls, sendbase, recvbase, send, recv,
                   recv_bytes, recv_after_local, NULL, 0, NULL, NULL, sz_local, usz_compact,
                   usz_global);
}

/*
 * Sec. IV-B and Algorithm 2: the local phase of Algorithm 3 followed by the
 * staggered inter-group exchange, one block per step, block_count steps per
 * batch.  K_out[1] = Q*(N-1) steps; *batches_out = batches that move anything.
 * Round rows of the global level carry RS_X = gi and RS_Z = gr.
 */
int oracle_tuna_hier_staggered(int Q, int N, int rl, int block_count, int elem,
                               const int64_t *counts, const int64_t *sdispls,
                               const int64_t *rdispls, const int64_t *sendbase,
                               const int64_t *recvbase, const uint8_t *send, uint8_t *recv,
                               int64_t recv_bytes, uint8_t *recv_after_local, int64_t *rounds,
                               int rounds_cap, int *K_out, int *batches_out) {
  if (block_count < 1) return ORACLE_EARG;
  return hier_impl(Q, N, rl, 2, block_count, elem, counts, sdispls, rdispls, sendbase, recvbase,
                   send, recv, recv_bytes, recv_after_local, rounds, rounds_cap, K_out,
                   batches_out, NULL, NULL, NULL);
}

/*
 * Not in the paper.  Counts and displacements are in rows of row_bytes bytes.
 * Row j of the (virtual) packed send buffer is row gather[j] of `in` (NULL: j
 * itself); row j of the (virtual) receive buffer lands in row scatter[j] of `out`
 * (NULL: j itself).  For every pair (s, d) and k < counts[s][d]:
 *   out[scatter[recvbase[d] + rdispls[d][s] + k]] = in[gather[sendbase[s] + sdispls[s][d] + k]].
 * Rows of `out` that no block reaches are left untouched.  Indices outside
 * [0, in_rows) / [0, out_rows) are an argument error.
 */
int oracle_rows_alltoallv(int P, int64_t row_bytes, const int64_t *counts, const int64_t *sdispls,
                          const int64_t *rdispls, const int64_t *sendbase,
                          const int64_t *recvbase, const int64_t *gather, const int64_t *scatter,
                          const uint8_t *in, int64_t in_rows, uint8_t *out, int64_t out_rows) {
  if (P < 1 || row_bytes < 1) return ORACLE_EARG;
  for (int s = 0; s < P; s++)
    for (int d = 0; d < P; d++) {
      int64_t n = counts[(int64_t)s * P + d];
      if (n < 0) return ORACLE_EARG;
      for (int64_t k = 0; k < n; k++) {
        int64_t js = sendbase[s] + sdispls[(int64_t)s * P + d] + k;
        int64_t jr = recvbase[d] + rdispls[(int64_t)d * P + s] + k;
        int64_t from = gather ? gather[js] : js;
        int64_t to = scatter ? scatter[jr] : jr;
        if (from < 0 || from >= in_rows || to < 0 || to >= out_rows) return ORACLE_EARG;
        memcpy(out + to * row_bytes, in + from * row_bytes, (size_t)row_bytes);
      }
    }
  return ORACLE_OK;
}
