// Plan kernels: the count-metadata exchange (Sec. III-B of the paper), the
// segmented exclusive prefix sums that turn block sizes into displacements
// (Sec. III-B/C), placement, work partition and the self-check.  Device code only;
// included by the translation units that launch these kernels.
#ifndef TUNA_PLAN_KERNELS_CUH
#define TUNA_PLAN_KERNELS_CUH

#include "tuna_internal.h"

namespace {

// ------------------------------------------------------------------ device helpers

__device__ __forceinline__ int64_t pad16(int64_t v) { return (v + (TUNA_ALIGN - 1)) & ~(int64_t)(TUNA_ALIGN - 1); }

// Compact index of offset v among the offsets whose digit (v / stride) % radix is
// non-zero, ascending.  Only called for such v.
__device__ __forceinline__ int64_t compact_of(int64_t v, int64_t stride, int radix) {
  const unsigned sr = (unsigned)stride * (unsigned)radix;  // at most P * radix < 2^31: 32-bit division
  const unsigned hi = (unsigned)v / sr;
  const int64_t rem = v - (int64_t)hi * sr;  // z*stride + lo
  return (int64_t)hi * (radix - 1) * stride + (rem - stride);
}

// Sharded plans: does this GPU hold rank p, and where does rank p receive.
__device__ __forceinline__ bool resident(const TunaTopo &t, int p) {
  return t.shard_n == 0 || p / t.Q == t.shard_me;
}
__device__ __forceinline__ int64_t recv_loc(const TunaTopo &t, int p, int64_t off) {
  return TUNA_LOC(t.shard_n ? TUNA_BUF_PEER0 + p / t.Q : TUNA_BUF_RECV, off);
}

struct PhaseDev {
  int level, radix, count;
  int64_t stride, moving, per_rank, finals;
};

// Row position of a moving slot among the blocks its rank receives in a phase
// (slot order), and the descriptor it maps to: the first `finals` positions of
// every rank's row are the blocks that have arrived (DELIVER list, `finals` per
// rank), the others travel on (KEEP list, per_rank - finals per rank).
__device__ __forceinline__ int64_t row_position(const TunaTopo &t, const PhaseDev &ph, int io, int jo) {
  return ph.level == 0 ? (int64_t)io * ph.moving + compact_of(jo, ph.stride, ph.radix)
                       : compact_of(io, ph.stride, ph.radix) * t.Q + jo;
}

// A plan's first phase finds every block where its owner put it: sizes and locations
// then follow from the layout itself, and the two tables need not exist yet.
struct TunaFirst {
  const int64_t *counts, *sdispls, *sendbase;  // all null from the second phase on
};
__device__ __forceinline__ int dest_of(const TunaTopo &t, int p, int sigma) {
  const int n = p / t.Q, q = p % t.Q, io = sigma / t.Q, jo = sigma % t.Q;
  return (n + io - (n + io >= t.N ? t.N : 0)) * t.Q + (q + jo - (q + jo >= t.Q ? t.Q : 0));
}
__device__ __forceinline__ int64_t first_size(const TunaTopo &t, const TunaFirst &f, int p, int sigma) {
  return f.counts[(int64_t)p * t.P + dest_of(t, p, sigma)] * t.elem;
}
__device__ __forceinline__ int64_t first_loc(const TunaTopo &t, const TunaFirst &f, int p, int sigma) {
  return TUNA_LOC(TUNA_BUF_SEND, (f.sendbase[p] + f.sdispls[(int64_t)p * t.P + dest_of(t, p, sigma)]) * t.elem);
}

// Initial tables (before any phase): every block is in its owner's send region
// (sz and loc may be null: a plan whose first phase is a digit phase works them out itself).
// Also fills the direct list (receive-side order (d, s)) and the self entries of
// the rotation list.
__global__ void tuna_init_tables_kernel(TunaTopo t, const int64_t *__restrict__ counts,
                                        const int64_t *__restrict__ sdispls,
                                        const int64_t *__restrict__ rdispls,
                                        const int64_t *__restrict__ sendbase,
                                        const int64_t *__restrict__ recvbase, int64_t *sz,
                                        int64_t *loc, int64_t *dir_len, int64_t *dir_src,
                                        int64_t *dir_dst, int64_t *rot_len, int64_t *rot_src,
                                        int64_t *rot_dst, int rot_dense) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t PP = (int64_t)t.P * t.P;
  if (idx >= PP) return;
  const int p = (int)((unsigned)idx / (unsigned)t.P), sigma = (int)((unsigned)idx % (unsigned)t.P);  // (P * P < 2^31)
  if (!sz && !dir_len && sigma != 0) return;  // only the self blocks are left to describe
  const int n = p / t.Q, q = p % t.Q, io = sigma / t.Q, jo = sigma % t.Q;
  const int dest = (n + io - (n + io >= t.N ? t.N : 0)) * t.Q + (q + jo - (q + jo >= t.Q ? t.Q : 0));
  const int64_t bytes = counts[(int64_t)p * t.P + dest] * t.elem;
  const int64_t sloc = TUNA_LOC(TUNA_BUF_SEND, (sendbase[p] + sdispls[(int64_t)p * t.P + dest]) * t.elem);
  if (sz) {
    sz[idx] = bytes;
    loc[idx] = sloc;
  }
  // direct list entry (d = p as receiver, s = sigma as source index)
  if (dir_len) {
    const int d = p, s = sigma;
    dir_len[idx] = counts[(int64_t)s * t.P + d] * t.elem;
    dir_src[idx] = TUNA_LOC(TUNA_BUF_SEND, (sendbase[s] + sdispls[(int64_t)s * t.P + d]) * t.elem);
    dir_dst[idx] = TUNA_LOC(TUNA_BUF_RECV, (recvbase[d] + rdispls[(int64_t)d * t.P + s]) * t.elem);
  }
  if (sigma == 0) {
    const int64_t r = rot_dense ? idx : p;
    rot_len[r] = resident(t, p) ? bytes : 0;  // (a sharded plan copies its own ranks' self blocks only)
    rot_src[r] = sloc;
    rot_dst[r] = recv_loc(t, p, (recvbase[p] + rdispls[(int64_t)p * t.P + p]) * t.elem);
  }
}

// Count-metadata exchange of one digit phase: the receiver (p', sigma) of every
// moving slot learns the size of the block its partner holds, and where the
// partner keeps it.  Non-moving slots keep their size.  Also accumulates the
// per-round byte totals (round z = the slots whose digit equals z).  sz_next is
// null in a plan's last phase: nothing reads the size table after it.
__global__ void tuna_meta_exchange_kernel(TunaTopo t, PhaseDev ph, TunaFirst first,
                                          const int64_t *__restrict__ sz_cur,
                                          const int64_t *__restrict__ loc_cur, int64_t *sz_next,
                                          int64_t *keep_len, int64_t *keep_src, int64_t *del_len,
                                          int64_t *del_src, unsigned long long *round_bytes) {
  extern __shared__ unsigned long long s_hist[];
  const bool use_smem = ph.radix <= 4096;
  if (use_smem) {
    for (int i = threadIdx.x; i < ph.radix; i += blockDim.x) s_hist[i] = 0;
    __syncthreads();
  }
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t PP = (int64_t)t.P * t.P;
  unsigned long long add = 0;  // bytes this thread's slot moves in round add_to (0: none)
  int add_to = 0;
  if (idx < PP) {
    const int p = (int)((unsigned)idx / (unsigned)t.P), sigma = (int)((unsigned)idx % (unsigned)t.P);  // (P * P < 2^31)
    const int n = p / t.Q, q = p % t.Q, io = sigma / t.Q, jo = sigma % t.Q;
    const int v = ph.level == 0 ? jo : io;
    const int dig = (int)(((unsigned)v / (unsigned)ph.stride) % (unsigned)ph.radix);
    if (dig == 0) {
      if (sz_next) sz_next[idx] = first.counts ? first_size(t, first, p, sigma) : sz_cur[idx];
    } else {
      const int dist = dig * (int)ph.stride;  // below Q (level 0) or N (level 1): a wrap is one addition
      int qs = q, ns = n;
      if (ph.level == 0) {
        qs -= dist;
        if (qs < 0) qs += t.Q;
      } else {
        ns -= dist;
        if (ns < 0) ns += t.N;
      }
      const int sender = ns * t.Q + qs;
      const int64_t c = row_position(t, ph, io, jo);
      const int64_t size = first.counts ? first_size(t, first, sender, sigma) : sz_cur[(int64_t)sender * t.P + sigma];
      const int64_t where = first.counts ? first_loc(t, first, sender, sigma) : loc_cur[(int64_t)sender * t.P + sigma];
      if (sz_next) sz_next[idx] = size;
      // sharded plans list a block only on the GPU that moves it: the receiver's in a
      // local phase (both ranks are there), the sender's in the global phase (a push)
      const int64_t bytes = resident(t, ph.level == 0 ? p : sender) ? size : 0;
      if (c < ph.finals) {
        const int64_t e = (int64_t)p * ph.finals + c;
        del_len[e] = bytes;
        del_src[e] = where;
      } else {
        const int64_t e = (int64_t)p * (ph.per_rank - ph.finals) + (c - ph.finals);
        keep_len[e] = bytes;
        keep_src[e] = where;
      }
      add = (unsigned long long)bytes;
      add_to = dig;
    }
  }
  // per-round byte counters.  The lanes of a warp often share the digit (slots of one
  // group, or a run of `stride` slots): they then add once, not 32 times to one address.
  {
    const int first = __shfl_sync(0xffffffffu, add_to, 0);
    if (__all_sync(0xffffffffu, add_to == first)) {
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) add += __shfl_xor_sync(0xffffffffu, add, d);
      if ((threadIdx.x & 31) != 0) add = 0;
    }
    if (add > 0 && add_to > 0) {
      if (use_smem)
        atomicAdd(&s_hist[add_to], add);
      else
        atomicAdd(&round_bytes[add_to], add);
    }
  }
  if (use_smem) {
    __syncthreads();
    for (int i = threadIdx.x; i < ph.radix; i += blockDim.x)
      if (s_hist[i]) atomicAdd(&round_bytes[i], s_hist[i]);
  }
}

// The same exchange for a level-0 phase whose radix is at least Q (one phase moves
// every local offset jo >= 1 once, from rank (n, q - jo) to rank (n, q); a flat plan
// with radix >= P is the case N = 1).  The general kernel would read the two tables
// along anti-diagonals, one 32-byte sector per value.  Here a CTA takes, for one
// group n and one destination group offset io, a 32 x 32 tile (sender's local id,
// jo): it reads the tile along rows and writes it out by receiver, where each
// receiver's slots are again consecutive; a round's bytes are summed per tile
// column first.  Grid: (tiles of a Q x Q square, N, N), CTAs of 32 x 8 threads.
__global__ void tuna_meta_exchange_diag_kernel(TunaTopo t, PhaseDev ph, TunaFirst first,
                                               const int64_t *__restrict__ sz_cur,
                                               const int64_t *__restrict__ loc_cur, int64_t *sz_next,
                                               int64_t *keep_len, int64_t *keep_src, int64_t *del_len,
                                               int64_t *del_src, unsigned long long *round_bytes) {
  __shared__ int64_t s_sz[32][32], s_loc[32][32];
  const int P = t.P, Q = t.Q, tx = threadIdx.x, ty = threadIdx.y;
  const int tiles = (Q + 31) / 32;
  const int g0 = ((int)blockIdx.x % tiles) * 32, s0 = ((int)blockIdx.x / tiles) * 32;  // first jo, first sender id
  const int io = blockIdx.y, n = blockIdx.z;
  const bool listed = t.shard_n == 0 || n == t.shard_me;  // (sharded plans: only the own group's blocks get a length)
  const int64_t row0 = (int64_t)n * Q;       // first rank of the group
  const int col0 = io * Q;                   // first slot of the destination group offset
  for (int j = ty; j < 32; j += 8) {
    const int sd = s0 + j, g = g0 + tx;
    const bool in = sd < Q && g < Q;
    if (first.counts) {
      s_sz[j][tx] = in ? first_size(t, first, (int)row0 + sd, col0 + g) : 0;
      s_loc[j][tx] = in ? first_loc(t, first, (int)row0 + sd, col0 + g) : 0;
    } else {
      s_sz[j][tx] = in ? sz_cur[(row0 + sd) * P + col0 + g] : 0;
      s_loc[j][tx] = in ? loc_cur[(row0 + sd) * P + col0 + g] : 0;
    }
  }
  __syncthreads();
  if (ty == 0 && g0 + tx >= 1 && g0 + tx < Q) {  // round z = jo: bytes sent by this tile's senders
    int64_t sum = 0;
#pragma unroll 8
    for (int j = 0; j < 32; j++) sum += s_sz[j][tx];
    if (sum > 0 && listed) atomicAdd(&round_bytes[g0 + tx], (unsigned long long)sum);
  }
  for (int pr = ty; pr < 63; pr += 8) {  // receivers s0 + g0 + pr (mod Q): a diagonal of the tile each
    const int sr = pr - tx;
    if (sr < 0 || sr >= 32) continue;
    const int sd = s0 + sr, g = g0 + tx;
    if (sd >= Q || g >= Q) continue;
    int q = sd + g;
    if (q >= Q) q -= Q;
    const int64_t p = row0 + q;
    int64_t bytes = s_sz[sr][tx];
    const int64_t where = s_loc[sr][tx];
    if (sz_next) sz_next[p * P + col0 + g] = bytes;  // (jo = 0 never moves in this phase: sender and receiver are the same rank)
    if (g == 0) continue;
    if (!listed) bytes = 0;
    const int64_t c = (int64_t)io * ph.moving + (g - 1);  // position among the blocks the rank receives, in slot order
    if (c < ph.finals) {
      const int64_t e = p * ph.finals + c;
      del_len[e] = bytes;
      del_src[e] = where;
    } else {
      const int64_t e = p * (ph.per_rank - ph.finals) + (c - ph.finals);
      keep_len[e] = bytes;
      keep_src[e] = where;
    }
  }
}

// Staggered inter-group exchange (Sec. IV-B, Algorithm 2), one batch: the steps
// ii in [lo, hi) of the index ii = gi*Q + gr, gi >= 1.  In step (gi, gr) rank
// (n, q) receives, from rank ((n + gi) mod N, q), the one block whose original
// owner is ((n + gi) mod N, gr).  Every such block has arrived: descriptor
// e = p*(hi - lo) + (ii - lo) of the batch's DELIVER list gets its size, where the
// sender keeps it, and its place in the receive buffer.  step_bytes[ii] sums the
// bytes of step ii over all ranks.
__global__ void tuna_stagger_batch_kernel(TunaTopo t, int lo, int hi,
                                          const int64_t *__restrict__ sz_cur,
                                          const int64_t *__restrict__ loc_cur,
                                          const int64_t *__restrict__ rdispls,
                                          const int64_t *__restrict__ recvbase, int64_t *del_len,
                                          int64_t *del_src, int64_t *del_dst,
                                          unsigned long long *step_bytes) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int m = hi - lo;
  if (idx >= (int64_t)t.P * m) return;
  const int p = (int)(idx / m), ii = lo + (int)(idx % m);
  const int n = p / t.Q, q = p % t.Q, gi = ii / t.Q, gr = ii % t.Q;
  const int nsrc = (n + gi) % t.N;
  const int sender = nsrc * t.Q + q, origin = nsrc * t.Q + gr;
  // the slot of that block, in offset coordinates: group offset from its owner's
  // group to this one, local offset from its owner to this rank
  const int sigma = ((t.N - gi) % t.N) * t.Q + (q - gr + t.Q) % t.Q;
  const int64_t bytes = sz_cur[(int64_t)sender * t.P + sigma];
  del_len[idx] = bytes;
  del_src[idx] = loc_cur[(int64_t)sender * t.P + sigma];
  del_dst[idx] = TUNA_LOC(TUNA_BUF_RECV, (recvbase[p] + rdispls[(int64_t)p * t.P + origin]) * t.elem);
  if (bytes > 0) atomicAdd(&step_bytes[ii], (unsigned long long)bytes);
}

// Row list of the exchange with a gather in front and a scatter behind (no
// counterpart in the paper): one descriptor per row.  One warp per block (d, s);
// row k of the block is row sendbase[s] + sdispls[s][d] + k of the packed send
// layout and row recvbase[d] + rdispls[d][s] + k of the receive layout; the maps
// (identity when null) turn these into rows of the caller's two buffers.
// row_start[d*P + s] = rows of all blocks before (d, s) in receive-side order.
__global__ void tuna_rows_list_kernel(int P, int64_t row_bytes, const int64_t *__restrict__ counts,
                                      const int64_t *__restrict__ sdispls,
                                      const int64_t *__restrict__ rdispls,
                                      const int64_t *__restrict__ sendbase,
                                      const int64_t *__restrict__ recvbase,
                                      const int64_t *__restrict__ row_start,
                                      const int64_t *__restrict__ gather,
                                      const int64_t *__restrict__ scatter, int64_t in_rows,
                                      int64_t out_rows, int64_t n_rows, int64_t *len, int64_t *pos,
                                      int64_t *src, int64_t *dst) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  const int64_t stride = pad16(row_bytes) + 16;  // DELIVER spacing of equal-sized blocks
  if (w == 0 && lane == 0) pos[n_rows] = n_rows * stride;
  if (w >= (int64_t)P * P) return;
  const int d = (int)(w / P), s = (int)(w % P);
  const int64_t c = counts[(int64_t)s * P + d];
  const int64_t js = sendbase[s] + sdispls[(int64_t)s * P + d];
  const int64_t jr = recvbase[d] + rdispls[(int64_t)d * P + s];
  const int64_t e0 = row_start[w];
  for (int64_t k = lane; k < c; k += 32) {
    const int64_t from = gather ? gather[js + k] : js + k;
    const int64_t to = scatter ? scatter[jr + k] : jr + k;
    const int64_t e = e0 + k;
    len[e] = row_bytes;
    pos[e] = e * stride;
    // a row outside its buffer gets a location that the range check that follows
    // rejects (the wrong buffer tag) instead of an offset that could wrap around
    src[e] = (from < 0 || from >= in_rows) ? TUNA_LOC(TUNA_BUF_RECV, 0) : TUNA_LOC(TUNA_BUF_SEND, from * row_bytes);
    dst[e] = (to < 0 || to >= out_rows) ? TUNA_LOC(TUNA_BUF_SEND, 0) : TUNA_LOC(TUNA_BUF_RECV, to * row_bytes);
  }
}

// Segmented exclusive prefix sum, one warp per segment, warp-shuffle scan over
// 128-wide tiles (four values per lane) with a running carry.  MODE 0 sums the values as they are; MODE 1
// (KEEP lists) rounds every value up to 16 first; MODE 2 (DELIVER lists) also
// adds 16 spare bytes behind every non-zero value.  seg_total[s] receives the
// segment's sum, seg_raw[s] (optional) the sum of the unmodified values.
template <int MODE>
__device__ __forceinline__ void segscan_body(const int64_t *__restrict__ val, int64_t *out,
                                             int64_t *seg_total, int64_t *seg_raw, int64_t seglen,
                                             int64_t nseg) {
  const int64_t w = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (w >= nseg) return;
  int64_t carry = 0, raw = 0;
  const int64_t *v = val + w * seglen;
  int64_t *o = out + w * seglen;
  // tiles of 128: every lane takes four consecutive values, sums them in registers,
  // and only the lanes' sums go through the shuffle scan
  constexpr int kPer = 4;
  for (int64_t base = 0; base < seglen; base += 32 * kPer) {
    const int64_t i0 = base + lane * kPer;
    int64_t x[kPer], sum = 0;
#pragma unroll
    for (int k = 0; k < kPer; k++) {
      int64_t y = i0 + k < seglen ? v[i0 + k] : 0;
      raw += y;
      if (MODE >= 1) y = pad16(y);
      if (MODE == 2 && y > 0) y += 16;
      x[k] = y;
      sum += y;
    }
    int64_t incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int64_t y = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += y;
    }
    int64_t run = carry + incl - sum;  // exclusive prefix of this lane's first value
#pragma unroll
    for (int k = 0; k < kPer; k++) {
      if (i0 + k < seglen) o[i0 + k] = run;
      run += x[k];
    }
    carry += __shfl_sync(0xffffffffu, incl, 31);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) raw += __shfl_xor_sync(0xffffffffu, raw, d);
  if (lane == 0) {
    seg_total[w] = carry;
    if (seg_raw) seg_raw[w] = raw;
  }
}

template <int MODE>
__global__ void tuna_segscan_kernel(const int64_t *__restrict__ val, int64_t *out,
                                    int64_t *seg_total, int64_t *seg_raw, int64_t seglen,
                                    int64_t nseg) {
  segscan_body<MODE>(val, out, seg_total, seg_raw, seglen, nseg);
}

// One list's scan as the kernels below take it.
struct TunaScanArgs {
  const int64_t *val;
  int64_t *out, *seg_total, *seg_raw, *seg_base;
  int64_t seglen, nseg;
  int64_t *scal, *wbase;
  int uses_work;
  int64_t *pos_end;
};

// The two lists of a digit phase in one launch: blockIdx.y = 0 scans the KEEP list
// (lengths rounded up to 16), blockIdx.y = 1 the DELIVER list (16 spare bytes more).
__global__ void tuna_segscan_pair_kernel(TunaScanArgs keep, TunaScanArgs del) {
  if (blockIdx.y == 0) {
    if (keep.seglen > 0) segscan_body<1>(keep.val, keep.out, keep.seg_total, keep.seg_raw, keep.seglen, keep.nseg);
  } else {
    if (del.seglen > 0) segscan_body<2>(del.val, del.out, del.seg_total, del.seg_raw, del.seglen, del.nseg);
  }
}

// Exclusive scan of the nseg segment totals (one CTA), giving every segment's
// base in the list's stream.  scal[0] = stream bytes, scal[1] = bytes moved.
// If wbase is given, wbase[1] = wbase[0] + (stream bytes rounded up to 256),
// or wbase[0] when the phase keeps nothing in the workspace.
__device__ __forceinline__ void segbase_body(const int64_t *__restrict__ seg_total,
                                             const int64_t *__restrict__ seg_raw, int64_t *seg_base,
                                             int64_t nseg, int64_t *scal, int64_t *wbase, int uses_work,
                                             int64_t *pos_end, int spaced = 0) {
  // (spaced: the values are block lengths, one block per segment: each is rounded up
  // to 16 and given 16 spare bytes here, and seg_base is the list's position array)
  __shared__ int64_t s_warp[32];
  __shared__ int64_t s_carry;
  __shared__ int64_t s_raw[32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  if (threadIdx.x == 0) s_carry = 0;
  int64_t raw = 0;
  __syncthreads();
  for (int64_t base = 0; base < nseg; base += blockDim.x) {
    const int64_t i = base + threadIdx.x;
    int64_t x = i < nseg ? seg_total[i] : 0;
    if (spaced) {
      raw += x;
      x = x > 0 ? pad16(x) + 16 : 0;
    } else if (seg_raw && i < nseg) {
      raw += seg_raw[i];
    }
    int64_t incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int64_t y = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += y;
    }
    if (lane == 31) s_warp[warp] = incl;
    __syncthreads();
    int64_t woff = 0;
    for (int k = 0; k < warp; k++) woff += s_warp[k];
    const int64_t carry = s_carry;
    if (i < nseg) seg_base[i] = carry + woff + incl - x;
    __syncthreads();
    if (threadIdx.x == blockDim.x - 1) s_carry = carry + woff + incl;
    __syncthreads();
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) raw += __shfl_xor_sync(0xffffffffu, raw, d);
  if (lane == 0) s_raw[warp] = raw;
  __syncthreads();
  if (threadIdx.x == 0) {
    int64_t r = 0;
    for (int k = 0; k < nw; k++) r += s_raw[k];
    scal[0] = s_carry;
    scal[1] = r;
    if (pos_end) *pos_end = s_carry;  // pos[n]: one past the last block
    if (wbase) wbase[1] = wbase[0] + (uses_work ? ((s_carry + 255) & ~(int64_t)255) : 0);
  }
}

__global__ void tuna_segbase_kernel(const int64_t *__restrict__ seg_total,
                                    const int64_t *__restrict__ seg_raw, int64_t *seg_base,
                                    int64_t nseg, int64_t *scal, int64_t *wbase, int uses_work,
                                    int64_t *pos_end, int spaced) {
  segbase_body(seg_total, seg_raw, seg_base, nseg, scal, wbase, uses_work, pos_end, spaced);
}

// The same for the two lists of a digit phase: CTA 0 the KEEP list, CTA 1 the DELIVER list.
__global__ void tuna_segbase_pair_kernel(TunaScanArgs keep, TunaScanArgs del) {
  if (blockIdx.x == 0)
    segbase_body(keep.seg_total, keep.seg_raw, keep.seg_base, keep.seglen > 0 ? keep.nseg : 0, keep.scal,
                 keep.wbase, keep.uses_work, keep.pos_end);
  else
    segbase_body(del.seg_total, del.seg_raw, del.seg_base, del.seglen > 0 ? del.nseg : 0, del.scal, del.wbase,
                 del.uses_work, del.pos_end);
}

// pos[e] += base of its segment (turns per-rank scans into one stream position).
__global__ void tuna_add_base_kernel(int64_t *pos, const int64_t *__restrict__ seg_base,
                                     int64_t seglen, int64_t n) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e < n) pos[e] += seg_base[e / seglen];
}

// Second half of a digit phase, after the prefix sums: stream positions become
// global, every moving block gets its destination, and the location table for
// the next phase is written.  A block whose remaining digits are all zero has
// arrived: in direct-to-R mode it is in the DELIVER list and goes to its place in
// the receive buffer; in classic mode every block stays in the workspace and a
// rotation descriptor is recorded for the final reorder.
__global__ void tuna_place_kernel(TunaTopo t, PhaseDev ph, TunaFirst first, const int64_t *__restrict__ loc_cur,
                                  int64_t *loc_next, int64_t *keep_pos,
                                  const int64_t *__restrict__ keep_base,
                                  const int64_t *__restrict__ keep_len, int64_t *del_pos,
                                  const int64_t *__restrict__ del_base, int64_t *del_dst,
                                  const int64_t *__restrict__ wbase,
                                  const int64_t *__restrict__ rdispls,
                                  const int64_t *__restrict__ recvbase, int classic,
                                  int64_t *rot_len, int64_t *rot_src, int64_t *rot_dst) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t PP = (int64_t)t.P * t.P;
  if (idx >= PP) return;
  const int p = (int)((unsigned)idx / (unsigned)t.P), sigma = (int)((unsigned)idx % (unsigned)t.P);  // (P * P < 2^31)
  const int n = p / t.Q, q = p % t.Q, io = sigma / t.Q, jo = sigma % t.Q;
  const int v = ph.level == 0 ? jo : io;
  const int dig = (int)(((unsigned)v / (unsigned)ph.stride) % (unsigned)ph.radix);
  if (dig == 0) {
    if (loc_next) loc_next[idx] = first.counts ? first_loc(t, first, p, sigma) : loc_cur[idx];
    return;
  }
  const int64_t c = row_position(t, ph, io, jo);
  const unsigned sr = (unsigned)ph.stride * (unsigned)ph.radix;
  const bool fin = ph.level == 0 ? (io == 0 && (unsigned)jo < sr) : (unsigned)io < sr;
  const int origin = (n - io + (n < io ? t.N : 0)) * t.Q + (q - jo + (q < jo ? t.Q : 0));
  const int64_t rloc = recv_loc(t, p, (recvbase[p] + rdispls[(int64_t)p * t.P + origin]) * t.elem);
  if (c < ph.finals) {  // DELIVER list (only in direct-to-R mode; these blocks have arrived)
    const int64_t e = (int64_t)p * ph.finals + c;
    del_pos[e] += del_base[p];
    del_dst[e] = rloc;
    if (loc_next) loc_next[idx] = rloc;
  } else {
    const int64_t e = (int64_t)p * (ph.per_rank - ph.finals) + (c - ph.finals);
    const int64_t w = keep_pos[e] + keep_base[p];
    keep_pos[e] = w;
    const int64_t wloc = TUNA_LOC(TUNA_BUF_WORK, wbase[0] + w);
    if (loc_next) loc_next[idx] = wloc;
    if (fin && classic) {
      rot_len[idx] = keep_len[e];
      rot_src[idx] = wloc;
      rot_dst[idx] = rloc;
    }
  }
}

// First descriptor of every chunk: the last e with pos[e] <= c * chunk.  One more
// entry closes the table: the last descriptor that has any bytes (so that a tail
// of empty blocks behind it is not walked by the last chunk's CTA).
__global__ void tuna_chunk_index_kernel(const int64_t *__restrict__ pos, int64_t n, int64_t chunk,
                                        int64_t nchunks, int64_t total, int32_t *first) {
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c > nchunks) return;
  const int64_t target = c < nchunks ? c * chunk : total - 1;
  int64_t lo = 0, hi = n;  // first index with pos > target
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if (pos[mid] <= target)
      lo = mid + 1;
    else
      hi = mid;
  }
  first[c] = (int32_t)(lo > 0 ? lo - 1 : 0);
}

// The same for several lists in one launch (blockIdx.y picks the list; the lists'
// parameters travel in the kernel's arguments).
struct TunaChunkItem {
  const int64_t *pos;
  int32_t *first;
  int64_t n, chunk, nchunks, total;
};
constexpr int kChunkBatch = 32;
struct TunaChunkBatch {
  TunaChunkItem it[kChunkBatch];
};

__global__ void tuna_chunk_index_batch_kernel(const __grid_constant__ TunaChunkBatch b) {
  const TunaChunkItem &it = b.it[blockIdx.y];
  const int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (c > it.nchunks) return;
  const int64_t target = c < it.nchunks ? c * it.chunk : it.total - 1;
  int64_t lo = 0, hi = it.n;  // first index with pos > target
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if (it.pos[mid] <= target)
      lo = mid + 1;
    else
      hi = mid;
  }
  it.first[c] = (int32_t)(lo > 0 ? lo - 1 : 0);
}

// Self-check of a finished list: every descriptor must read inside its source
// buffer and write inside its destination.  The movers touch no other bytes than
// these ranges (plus the documented aligned over-read inside the source buffer),
// so a clean check bounds every access of the exchange.  Violations are counted.
__device__ __forceinline__ void check_list_body(const int64_t *__restrict__ len, const int64_t *__restrict__ pos,
                                                const int64_t *__restrict__ src, const int64_t *__restrict__ dst,
                                                int64_t n, const int64_t *__restrict__ extents,
                                                const int64_t *__restrict__ work_extent, int64_t keep_base_index,
                                                const int64_t *__restrict__ wbase, unsigned long long *violations,
                                                unsigned long long *unaligned_bytes,
                                                const int64_t *__restrict__ peer_extents = nullptr) {
  bool bad = false;
  int64_t skewed = 0;  // bytes of blocks whose source and destination differ modulo 16
  const int64_t send_extent = extents[0], recv_extent = extents[1];
  const int64_t wext = *work_extent, wb = wbase[keep_base_index];
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (int64_t)gridDim.x * blockDim.x) {
    // all of a descriptor's fields at once: one round trip to memory per descriptor
    const int64_t L = len[e], p0 = pos[e], p1 = pos[e + 1], s = src[e], d = dst ? dst[e] : 0;
    bad = bad || L < 0 || p1 < p0;
    if (L > 0) {
      const int sb = TUNA_LOC_BUF(s);
      const int64_t so = TUNA_LOC_OFF(s);
      const int64_t sext = sb == TUNA_BUF_SEND ? send_extent : (sb == TUNA_BUF_WORK ? wext : -1);
      bad = bad || so < 0 || so + L > sext;
      if (dst) {  // DELIVER: into the receive buffer (sharded plans: the receiving GPU's)
        const int db = TUNA_LOC_BUF(d);
        const int64_t dext = db == TUNA_BUF_RECV ? recv_extent
                                                 : (db >= TUNA_BUF_PEER0 && peer_extents ? peer_extents[db - TUNA_BUF_PEER0] : -1);
        bad = bad || TUNA_LOC_OFF(d) + L > dext;
        if (((so - TUNA_LOC_OFF(d)) & 15) != 0) skewed += L;
      } else {    // KEEP: at its stream position in the phase's workspace region
        const int64_t o = wb + p0;
        bad = bad || (o & (TUNA_ALIGN - 1)) != 0 || o + pad16(L) > wext || p1 - p0 != pad16(L);
        if ((so & 15) != 0) skewed += L;
      }
    }
  }
  if (bad) atomicAdd(violations, 1ULL);
  // one atomic per CTA of a bounded grid: a list of millions of blocks would
  // otherwise queue a hundred thousand of them on one address
  __shared__ int64_t s_part[32];
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) skewed += __shfl_xor_sync(0xffffffffu, skewed, d);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = skewed;
  __syncthreads();
  if (threadIdx.x < 32) {
    int64_t v = threadIdx.x < (blockDim.x + 31) / 32 ? s_part[threadIdx.x] : 0;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
    if (threadIdx.x == 0 && v > 0) atomicAdd(unaligned_bytes, (unsigned long long)v);
  }
}

__global__ void tuna_check_list_kernel(const int64_t *__restrict__ len, const int64_t *__restrict__ pos,
                                       const int64_t *__restrict__ src, const int64_t *__restrict__ dst,
                                       int64_t n, const int64_t *__restrict__ extents,
                                       const int64_t *__restrict__ work_extent, int64_t keep_base_index,
                                       const int64_t *__restrict__ wbase, unsigned long long *violations,
                                       unsigned long long *unaligned_bytes) {
  check_list_body(len, pos, src, dst, n, extents, work_extent, keep_base_index, wbase, violations, unaligned_bytes);
}

// All lists of a plan in one launch: blockIdx.y picks the list.
struct TunaCheckItem {
  const int64_t *len, *pos, *src, *dst;  // dst null: a KEEP list
  int64_t n;
  int64_t keep_base_index;  // KEEP lists: the phase, whose workspace offset is wbase[phase]
  int64_t id;               // slot of the list's skewed-byte counter behind violations[0]
};

__global__ void tuna_check_lists_kernel(const TunaCheckItem *__restrict__ items, const int64_t *__restrict__ extents,
                                        const int64_t *__restrict__ work_extent,
                                        const int64_t *__restrict__ wbase, unsigned long long *violations,
                                        const int64_t *__restrict__ peer_extents) {
  const TunaCheckItem it = items[blockIdx.y];
  if ((int64_t)blockIdx.x * blockDim.x >= it.n) return;  // (whole CTA: short lists need few of them)
  check_list_body(it.len, it.pos, it.src, it.dst, it.n, extents, work_extent, it.keep_base_index, wbase,
                  violations, violations + 1 + it.id, peer_extents);
}

// out = in^T, in 32 x 32 tiles through shared memory so that both the reads and the
// writes run along rows (grid: ceil(P/32) x ceil(P/32) CTAs of 32 x 8 threads).
// With `negatives`, entries below zero are counted there (counts that arrive in
// device memory are validated in this pass).
__global__ void tuna_transpose_kernel(const int64_t *__restrict__ in, int64_t *out, int P, int64_t *negatives) {
  __shared__ int64_t tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;  // the tile in[r0.., c0..]
  for (int j = threadIdx.y; j < 32; j += 8) {
    const int r = r0 + j, c = c0 + threadIdx.x;
    if (r < P && c < P) {
      const int64_t v = in[(int64_t)r * P + c];
      tile[j][threadIdx.x] = v;
      if (negatives && v < 0) atomicAdd(reinterpret_cast<unsigned long long *>(negatives), 1ULL);
    }
  }
  __syncthreads();
  for (int j = threadIdx.y; j < 32; j += 8) {
    const int r = c0 + j, c = r0 + threadIdx.x;  // out[r][c] = in[c][r]
    if (r < P && c < P) out[(int64_t)r * P + c] = tile[threadIdx.x][j];
  }
}

// Packed layout worked out on the device: both buffers extend over the sum of all
// counts (tot[0], in elements).
__global__ void tuna_packed_extents_kernel(const int64_t *__restrict__ tot, int elem, int64_t *extents) {
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    extents[0] = tot[0] * elem;
    extents[1] = tot[0] * elem;
    extents[2] = tot[0];
  }
}

// Sharded plans whose counts arrive in device memory: a GPU's regions are packed in
// rank order from offset 0 of ITS buffer, so the bases are running sums that start
// anew with every group of Q ranks.  base[p] = elements of the regions before rank p's
// on its GPU; group_total[n] = elements of GPU n's buffer.
__global__ void tuna_shard_bases_kernel(const int64_t *__restrict__ seg_total, int P, int Q, int64_t *base,
                                        int64_t *group_total) {
  const int p = blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= P) return;
  const int n = p / Q;
  int64_t sum = 0;
  for (int i = n * Q; i < p; i++) sum += seg_total[i];
  base[p] = sum;
  if (p == n * Q + Q - 1) group_total[n] = sum + seg_total[p];
}

// ... and the extents that follow from the GPUs' totals: this GPU's two buffers and the
// payload (extents[0..2], as for a plan on one GPU), every GPU's receive buffer for the
// self-check (peer_extent) and every GPU's send buffer for the host (send_extent), in bytes.
__global__ void tuna_shard_extents_kernel(const int64_t *__restrict__ send_total,
                                          const int64_t *__restrict__ recv_total, int N, int me, int elem,
                                          int64_t *extents, int64_t *peer_extent, int64_t *send_extent) {
  if (blockIdx.x != 0 || threadIdx.x != 0) return;
  int64_t all = 0;
  for (int n = 0; n < N; n++) {
    all += send_total[n];
    peer_extent[n] = recv_total[n] * elem;
    send_extent[n] = send_total[n] * elem;
  }
  extents[0] = send_total[me] * elem;
  extents[1] = recv_total[me] * elem;
  extents[2] = all;
}

}  // namespace

#endif
