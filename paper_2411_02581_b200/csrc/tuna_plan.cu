// Plan construction (count-metadata exchange + segmented prefix sums) and the
// C-ABI entry points.
//
// Device-side picture.  Rank p = n*Q + q (Q = l ranks per group, N = g groups;
// flat TuNA is N = 1).  Every rank names its P blocks by slot sigma = io*Q + jo,
// the block for rank (n+io mod N, q+jo mod Q): this is the paper's index-only
// rotation (Algorithm 1, the array I), no data moves.  A digit phase (level, x)
// with radix r moves every slot whose digit x of jo (level 0) or io (level 1) is
// z != 0 to the rank at distance +z*r^x on that level (Sec. III-A, Sec. IV).
// Two dense P x P tables follow the blocks through the phases:
//     sz[p][sigma]   size of the block rank p holds in that slot    (Sec. III-B:
//                    the per-round metadata message is the same rank shift
//                    applied to this table)
//     loc[p][sigma]  where its bytes are (send buffer or a workspace offset)
// and every phase emits a compact descriptor list in receive-side order whose
// destination offsets are exclusive prefix sums of the 16-byte-padded sizes
// (Sec. III-C's temporary buffer, sized exactly instead of by the maximum block).
#include <stdio.h>
#include <stdlib.h>
#include <string.h>
#include <unistd.h>

#include <algorithm>
#include <atomic>
#include <condition_variable>
#include <functional>
#include <mutex>
#include <new>
#include <thread>

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

// Initial tables (before any phase): every block is in its owner's send region.
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
  const int n = p / t.Q, q = p % t.Q, io = sigma / t.Q, jo = sigma % t.Q;
  const int dest = (n + io - (n + io >= t.N ? t.N : 0)) * t.Q + (q + jo - (q + jo >= t.Q ? t.Q : 0));
  const int64_t bytes = counts[(int64_t)p * t.P + dest] * t.elem;
  const int64_t sloc = TUNA_LOC(TUNA_BUF_SEND, (sendbase[p] + sdispls[(int64_t)p * t.P + dest]) * t.elem);
  sz[idx] = bytes;
  loc[idx] = sloc;
  // direct list entry (d = p as receiver, s = sigma as source index)
  if (dir_len) {
    const int d = p, s = sigma;
    dir_len[idx] = counts[(int64_t)s * t.P + d] * t.elem;
    dir_src[idx] = TUNA_LOC(TUNA_BUF_SEND, (sendbase[s] + sdispls[(int64_t)s * t.P + d]) * t.elem);
    dir_dst[idx] = TUNA_LOC(TUNA_BUF_RECV, (recvbase[d] + rdispls[(int64_t)d * t.P + s]) * t.elem);
  }
  if (sigma == 0) {
    const int64_t r = rot_dense ? idx : p;
    rot_len[r] = bytes;
    rot_src[r] = sloc;
    rot_dst[r] = TUNA_LOC(TUNA_BUF_RECV, (recvbase[p] + rdispls[(int64_t)p * t.P + p]) * t.elem);
  }
}

// Count-metadata exchange of one digit phase: the receiver (p', sigma) of every
// moving slot learns the size of the block its partner holds, and where the
// partner keeps it.  Non-moving slots keep their size.  Also accumulates the
// per-round byte totals (round z = the slots whose digit equals z).
__global__ void tuna_meta_exchange_kernel(TunaTopo t, PhaseDev ph, const int64_t *__restrict__ sz_cur,
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
      sz_next[idx] = sz_cur[idx];
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
      const int64_t bytes = sz_cur[(int64_t)sender * t.P + sigma];
      const int64_t where = loc_cur[(int64_t)sender * t.P + sigma];
      sz_next[idx] = bytes;
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
__global__ void tuna_meta_exchange_diag_kernel(TunaTopo t, PhaseDev ph, const int64_t *__restrict__ sz_cur,
                                               const int64_t *__restrict__ loc_cur, int64_t *sz_next,
                                               int64_t *keep_len, int64_t *keep_src, int64_t *del_len,
                                               int64_t *del_src, unsigned long long *round_bytes) {
  __shared__ int64_t s_sz[32][32], s_loc[32][32];
  const int P = t.P, Q = t.Q, tx = threadIdx.x, ty = threadIdx.y;
  const int tiles = (Q + 31) / 32;
  const int g0 = ((int)blockIdx.x % tiles) * 32, s0 = ((int)blockIdx.x / tiles) * 32;  // first jo, first sender id
  const int io = blockIdx.y, n = blockIdx.z;
  const int64_t row0 = (int64_t)n * Q;       // first rank of the group
  const int col0 = io * Q;                   // first slot of the destination group offset
  for (int j = ty; j < 32; j += 8) {
    const int sd = s0 + j, g = g0 + tx;
    const bool in = sd < Q && g < Q;
    s_sz[j][tx] = in ? sz_cur[(row0 + sd) * P + col0 + g] : 0;
    s_loc[j][tx] = in ? loc_cur[(row0 + sd) * P + col0 + g] : 0;
  }
  __syncthreads();
  if (ty == 0 && g0 + tx >= 1 && g0 + tx < Q) {  // round z = jo: bytes sent by this tile's senders
    int64_t sum = 0;
#pragma unroll 8
    for (int j = 0; j < 32; j++) sum += s_sz[j][tx];
    if (sum > 0) atomicAdd(&round_bytes[g0 + tx], (unsigned long long)sum);
  }
  for (int pr = ty; pr < 63; pr += 8) {  // receivers s0 + g0 + pr (mod Q): a diagonal of the tile each
    const int sr = pr - tx;
    if (sr < 0 || sr >= 32) continue;
    const int sd = s0 + sr, g = g0 + tx;
    if (sd >= Q || g >= Q) continue;
    int q = sd + g;
    if (q >= Q) q -= Q;
    const int64_t p = row0 + q;
    const int64_t bytes = s_sz[sr][tx], where = s_loc[sr][tx];
    sz_next[p * P + col0 + g] = bytes;  // (jo = 0 never moves in this phase: sender and receiver are the same rank)
    if (g == 0) continue;
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
__global__ void tuna_place_kernel(TunaTopo t, PhaseDev ph, const int64_t *__restrict__ loc_cur,
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
    loc_next[idx] = loc_cur[idx];
    return;
  }
  const int64_t c = row_position(t, ph, io, jo);
  const unsigned sr = (unsigned)ph.stride * (unsigned)ph.radix;
  const bool fin = ph.level == 0 ? (io == 0 && (unsigned)jo < sr) : (unsigned)io < sr;
  const int origin = (n - io + (n < io ? t.N : 0)) * t.Q + (q - jo + (q < jo ? t.Q : 0));
  const int64_t rloc =
      TUNA_LOC(TUNA_BUF_RECV, (recvbase[p] + rdispls[(int64_t)p * t.P + origin]) * t.elem);
  if (c < ph.finals) {  // DELIVER list (only in direct-to-R mode; these blocks have arrived)
    const int64_t e = (int64_t)p * ph.finals + c;
    del_pos[e] += del_base[p];
    del_dst[e] = rloc;
    loc_next[idx] = rloc;
  } else {
    const int64_t e = (int64_t)p * (ph.per_rank - ph.finals) + (c - ph.finals);
    const int64_t w = keep_pos[e] + keep_base[p];
    keep_pos[e] = w;
    const int64_t wloc = TUNA_LOC(TUNA_BUF_WORK, wbase[0] + w);
    loc_next[idx] = wloc;
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
                                                unsigned long long *unaligned_bytes) {
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
      if (dst) {  // DELIVER: into the receive buffer
        bad = bad || TUNA_LOC_BUF(d) != TUNA_BUF_RECV || TUNA_LOC_OFF(d) + L > recv_extent;
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
                                        const int64_t *__restrict__ wbase, unsigned long long *violations) {
  const TunaCheckItem it = items[blockIdx.y];
  if ((int64_t)blockIdx.x * blockDim.x >= it.n) return;  // (whole CTA: short lists need few of them)
  check_list_body(it.len, it.pos, it.src, it.dst, it.n, extents, work_extent, it.keep_base_index, wbase,
                  violations, violations + 1 + it.id);
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

}  // namespace

// ------------------------------------------------------------------ the plan object

struct tuna_plan {
  TunaTopo topo{};
  int radix_l = 2, radix_g = 2;
  int block_count = 0;  // > 0: staggered inter-group exchange in batches of this many steps
  unsigned flags = 0;
  bool classic = false;
  int cuda_err = 0;
  int last_launches = 0;

  std::vector<TunaPhase> phases;
  std::vector<TunaList> keep;     // per phase: blocks that travel on (workspace)
  std::vector<TunaList> deliver;  // per phase: blocks that have arrived (receive buffer)
  TunaList rot, dir;
  // A flat direct-to-R plan with a single digit phase (radix >= P) delivers every
  // block in that phase: its DELIVER list and the self blocks together are the
  // direct exchange, so no separate direct list is built.
  bool dir_shared = false;
  bool no_direct = false;  // TUNA_FLAG_NO_DIRECT: no direct list at all (unless the phase's lists serve as one)
  // exchange of rows through a gather and a scatter map (tuna_plan_set_row_maps)
  TunaList rowsl;
  int64_t rows_cap = 0;          // descriptors allocated in rowsl
  int64_t *d_row_start = nullptr;
  int64_t rows_in_bytes = 0, rows_out_bytes = 0;
  bool rows_valid = false;

  struct Round {
    int level, x, z, phase;
    int64_t units, bytes;
    int64_t stat;  // index of its byte counter in the stats array
  };
  std::vector<Round> rounds;

  // host copies for validation
  // The count matrix on the host, for the checks at call time and as the source of
  // the upload: two buffers (pinned when that can be had), so that new counts are
  // validated and copied in one pass into the spare one and a rejected update
  // leaves the plan as it was.
  int64_t *h_counts = nullptr;  // the buffer that matches the device tables
  int64_t *h_buf[2] = {nullptr, nullptr};
  bool h_pinned = false;
  int h_cur = 0;
  std::vector<int64_t> h_sdispls, h_rdispls;
  bool have_sdispls = false, have_rdispls = false;
  bool h_counts_valid = true;   // false after an update from device counts, until they are read back
  bool tables_valid = false;    // false while an update is under way and after one that failed
  int64_t send_extent = 0, recv_extent = 0, payload = 0;  // bytes

  // device tables
  int64_t *d_counts = nullptr, *d_sdispls = nullptr, *d_rdispls = nullptr;
  int64_t *d_counts_buf[2] = {nullptr, nullptr};  // d_counts is one of them; an update fills the other
  bool counts_uploaded = false;  // the host pass already sent the counts to d_counts
  int64_t *d_sendbase = nullptr, *d_recvbase = nullptr;
  int64_t *d_sz[2] = {nullptr, nullptr}, *d_loc[2] = {nullptr, nullptr};
  int64_t *d_seg_total = nullptr, *d_seg_raw = nullptr, *d_seg_base = nullptr;
  int64_t *d_tmp = nullptr;      // P*P scratch (transpose)
  // The small tables an update reads back are slices of one allocation, so that one
  // copy into one pinned host buffer fetches them all.
  int64_t *d_readback = nullptr, *h_readback = nullptr;
  int64_t readback_words = 0;
  int64_t *d_scal = nullptr;     // per list: stream bytes, bytes moved
  int64_t *d_wbase = nullptr;    // phases + 1 workspace offsets
  int64_t *d_extents = nullptr;  // send extent, receive extent (bytes), total of the counts (elements),
                                 // number of negative counts seen
  unsigned long long *d_round_bytes = nullptr;
  int64_t stats_n = 0;
  int *d_error = nullptr;        // raised by a kernel whose bounded wait gave up
  unsigned long long *d_violations = nullptr;  // [0]: descriptors that failed the plan's self-check;
                                               // [1 + list id]: bytes of that list's blocks whose source
                                               // and destination differ modulo 16

  std::vector<int64_t> h_wbase;  // workspace offset of every phase's KEEP stream
  int64_t workspace_need = 0;
  char *workspace = nullptr;
  size_t workspace_bytes = 0;

  int64_t launch_count = 0;  // kernels launched by this plan since creation
  void *d_check_items = nullptr;    // the plan's lists as the self-check kernel takes them (fixed at creation)
  int n_check_items = 0;
  int64_t check_max_n = 0;
  cudaEvent_t in_flight = nullptr;  // end of the last exchange this plan enqueued (outside graph capture)
  bool in_flight_set = false;
  // An update's last kernels (the chunk tables) are not waited for on the host: an
  // event marks their end, and an exchange on another stream waits for it there.
  cudaEvent_t tables_ready = nullptr;
  bool tables_ready_set = false;
  cudaStream_t ready_waited = nullptr;  // the stream that is known to be ordered behind the event
  // The plan kernels of an update from device counts, captured once as a CUDA graph
  // (their arguments do not change from update to update) and replayed afterwards.
  cudaStream_t capture_stream = nullptr;
  cudaGraphExec_t tables_graph = nullptr;
  const int64_t *tables_graph_counts = nullptr;  // the count buffer the captured kernels read
  int64_t tables_graph_launches = 0;

  // optional per-launch timing (CUDA events on the caller's stream)
  bool timing = false;
  struct Stamp {
    int kind;
    int64_t bytes;
    cudaEvent_t a, b;
  };
  std::vector<Stamp> stamps;
  std::vector<cudaEvent_t> event_pool;
  double t_ms[TUNA_TIMER_KINDS] = {};
  int64_t t_launches[TUNA_TIMER_KINDS] = {};
  int64_t t_bytes[TUNA_TIMER_KINDS] = {};
};

namespace {

#define TUNA_CUDA(plan, call)                     \
  do {                                            \
    cudaError_t e_ = (call);                      \
    if (e_ != cudaSuccess) {                      \
      (plan)->cuda_err = (int)e_;                 \
      return TUNA_ERR_CUDA;                       \
    }                                             \
  } while (0)

// after a kernel launch: count it and check the launch status
#define TUNA_LAUNCHED(plan)                       \
  do {                                            \
    (plan)->launch_count++;                       \
    TUNA_CUDA(plan, cudaGetLastError());          \
  } while (0)

// An exchange reads the plan's tables until it ends; an update rewrites them.  Every
// exchange call marks its end on its stream, and an update waits for the mark.  A
// stream that is being captured gets no mark (an event recorded there could not be
// waited for later): replays of a captured exchange are the caller's to order.
int mark_in_flight(tuna_plan *pl, cudaStream_t st) {
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) {
    (void)cudaGetLastError();
    return TUNA_OK;
  }
  if (cap != cudaStreamCaptureStatusNone) return TUNA_OK;
  if (!pl->in_flight) TUNA_CUDA(pl, cudaEventCreateWithFlags(&pl->in_flight, cudaEventDisableTiming));
  TUNA_CUDA(pl, cudaEventRecord(pl->in_flight, st));
  pl->in_flight_set = true;
  return TUNA_OK;
}

int wait_in_flight(tuna_plan *pl) {
  if (pl->in_flight_set) {
    TUNA_CUDA(pl, cudaEventSynchronize(pl->in_flight));
    pl->in_flight_set = false;
  }
  if (pl->tables_ready_set) {  // (the previous update's chunk tables, possibly on another stream)
    TUNA_CUDA(pl, cudaEventSynchronize(pl->tables_ready));
    pl->tables_ready_set = false;
  }
  return TUNA_OK;
}

// End of an update: the tables are complete once everything enqueued on `st` so far has run.
int mark_tables_ready(tuna_plan *pl, cudaStream_t st) {
  if (!pl->tables_ready) TUNA_CUDA(pl, cudaEventCreateWithFlags(&pl->tables_ready, cudaEventDisableTiming));
  TUNA_CUDA(pl, cudaEventRecord(pl->tables_ready, st));
  pl->tables_ready_set = true;
  pl->ready_waited = st;  // work enqueued on the same stream is behind it already
  return TUNA_OK;
}

// Start of an exchange on `st`: order it behind the last update's kernels.
int await_tables(tuna_plan *pl, cudaStream_t st) {
  if (!pl->tables_ready_set || st == pl->ready_waited) return TUNA_OK;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) {
    (void)cudaGetLastError();
    cap = cudaStreamCaptureStatusNone;
  }
  if (cap != cudaStreamCaptureStatusNone) {  // a capture cannot wait for an event from outside: wait here
    TUNA_CUDA(pl, cudaEventSynchronize(pl->tables_ready));
    return TUNA_OK;
  }
  TUNA_CUDA(pl, cudaStreamWaitEvent(st, pl->tables_ready, 0));
  pl->ready_waited = st;
  return TUNA_OK;
}

cudaEvent_t take_event(tuna_plan *pl) {
  cudaEvent_t e = nullptr;
  if (!pl->event_pool.empty()) {
    e = pl->event_pool.back();
    pl->event_pool.pop_back();
  } else if (cudaEventCreate(&e) != cudaSuccess) {
    e = nullptr;
  }
  return e;
}

// Brackets one launch (or the plan kernels) with events when timing is on.
struct Timed {
  tuna_plan *pl;
  cudaStream_t st;
  tuna_plan::Stamp s{};
  bool on;
  Timed(tuna_plan *p, int kind, int64_t bytes, cudaStream_t stream) : pl(p), st(stream), on(p->timing) {
    if (!on) return;
    s.kind = kind;
    s.bytes = bytes;
    s.a = take_event(pl);
    s.b = take_event(pl);
    if (!s.a || !s.b) {
      on = false;
      return;
    }
    cudaEventRecord(s.a, st);
  }
  void stop() {
    if (!on) return;
    on = false;
    cudaEventRecord(s.b, st);
    pl->stamps.push_back(s);
  }
  ~Timed() { stop(); }
};

int64_t ipow64(int64_t r, int x) {
  int64_t v = 1;
  while (x-- > 0) v *= r;
  return v;
}

int num_digits(int count, int r) {
  int w = 0;
  int64_t pw = 1;
  while (pw < count) {
    pw *= r;
    w++;
  }
  return w;
}

int64_t count_digit(int count, int r, int x, int z) {  // offsets < count with digit x == z
  int64_t c = 0, stride = ipow64(r, x);
  for (int v = 0; v < count; v++) c += ((v / stride) % r) == z;
  return c;
}

template <class T>
cudaError_t dev_alloc(T **p, int64_t n) {
  return cudaMalloc((void **)p, (size_t)std::max<int64_t>(n, 1) * sizeof(T));
}

void free_list(TunaList &l) {
  cudaFree(l.len);
  cudaFree(l.pos);
  cudaFree(l.src);
  cudaFree(l.dst);
  cudaFree(l.chunk_first);
  l = TunaList();
}

int alloc_list(tuna_plan *pl, TunaList &l, int kind, int64_t n) {
  l.kind = kind;
  l.n = n;
  TUNA_CUDA(pl, dev_alloc(&l.len, n));
  TUNA_CUDA(pl, dev_alloc(&l.pos, n + 1));
  TUNA_CUDA(pl, dev_alloc(&l.src, n));
  if (kind == TUNA_LIST_DELIVER) TUNA_CUDA(pl, dev_alloc(&l.dst, n));
  return TUNA_OK;
}

int64_t env_i64(const char *name, int64_t dflt) {
  const char *s = getenv(name);
  if (!s || !*s) return dflt;
  return strtoll(s, nullptr, 10);
}

// Which kernel build runs a list.  Measured on the direct exchange (TB/s of read +
// write, large build / small build): blocks whose source and destination agree
// modulo 16 (plain vector copies) 2.86 / 3.58 at 64-byte blocks, 4.20 / 4.84 at
// 128 B, 5.37 / 5.22 at 256 B, 5.89 / 5.67 at 4 KiB, 6.40 / 6.07 at 128 KiB,
// 6.56 / 6.12 at 1 MiB; blocks that need the funnel-shift loads 2.38 / 2.83 at 128 B,
// 3.77 / 4.40 at 1 KiB, 4.23 / 4.93 at 32 KiB, 4.55 / 5.31 at 1 MiB.  So: the small
// build for lists of tiny blocks and for lists that are mostly skewed, whatever
// their block size; the large build otherwise.  Lists small enough to live in L2
// are latency-bound rather than DRAM-bound and also do better with the small
// build's higher occupancy (c3, 16 x 16 ranks, radix 16/2: 0.144 ms against 0.169 ms).
// Skewed lists of large blocks go back to the large build: a chunk inside one
// skewed block takes its own path there (one aligned load per vector, the
// neighbour's words by shuffle).  Measured, small / large build: 5.27 / 4.95 TB/s
// at 128 KiB mean block size, 5.29 / 5.36 at 256 KiB, 5.36 / 5.78 at 1 MiB,
// 5.53 / 6.22 at 4 MiB.
constexpr int64_t kSkewedLargeBlockBytes = 256 << 10;
constexpr int64_t kSmallBlockBytes = 256;
constexpr int64_t kSmallListBytes = 64 << 20;
constexpr int64_t kStaticSmallBlockBytes = 65536;  // the table-free entry point decides by size alone
constexpr int64_t kHostStagingBlockBytes = 2048;  // mean block below which host buffers are staged

// Bytes of stream per CTA.  Large build: 64 KiB, the best measured size for
// multi-MiB blocks (smaller chunks pay the per-chunk set-up more often, larger
// ones leave a longer tail); 128 KiB for blocks of 1 to 32 KiB (measured: 6.03 vs
// 5.89 TB/s at 4 KiB, 6.10 vs 5.96 at 16 KiB, 6.35 vs 6.00 on scattered 8 KiB
// rows).  Small build: 32 KiB, so that one batch of 256 descriptors covers a chunk
// of tiny blocks.  Small lists: fewer bytes per CTA, to fill the SMs.
int64_t pick_chunk(const TunaList &l) {
  const int64_t forced = env_i64(l.kind == TUNA_LIST_KEEP ? "TUNA_CHUNK_BYTES_KEEP" : "TUNA_CHUNK_BYTES_DELIVER", 0);
  if (forced >= 1024) return std::min<int64_t>((forced + 15) & ~(int64_t)15, TUNA_MAX_CHUNK_BYTES);
  const int64_t mean = l.n > 0 ? l.bytes / l.n : 0;
  const int64_t top = l.small_blocks ? 32768 : ((mean >= 1024 && mean <= 32768) ? 131072 : 65536);
  int64_t c = 8192;
  while (c < top && l.total / c > 148 * 32) c <<= 1;
  return c;
}

// With `batch`, the list's table is not computed here: its parameters are collected
// and launch_chunk_batch computes the tables of all collected lists in one launch.
struct ChunkCollector {
  TunaChunkBatch b;
  int n = 0;
  int64_t max_chunks = 0;
};

int launch_chunk_batch(tuna_plan *pl, ChunkCollector &cc, cudaStream_t st) {
  if (cc.n == 0) return TUNA_OK;
  const int th = 128;
  tuna_chunk_index_batch_kernel<<<dim3((unsigned)((cc.max_chunks + th) / th), cc.n), th, 0, st>>>(cc.b);
  TUNA_LAUNCHED(pl);
  cc.n = 0;
  cc.max_chunks = 0;
  return TUNA_OK;
}

int build_chunks(tuna_plan *pl, TunaList &l, cudaStream_t st, ChunkCollector *batch = nullptr) {
  l.small_blocks = l.n > 0 && (l.bytes / l.n < env_i64("TUNA_SMALL_BLOCK_BYTES", kSmallBlockBytes) ||
                               l.bytes < env_i64("TUNA_SMALL_LIST_BYTES", kSmallListBytes) ||
                               (2 * l.unaligned_bytes > l.bytes && l.bytes / l.n < kSkewedLargeBlockBytes &&
                                env_i64("TUNA_SKEWED_SMALL", 1) != 0));
  l.chunk = pick_chunk(l);
  l.nchunks = l.total > 0 ? (l.total + l.chunk - 1) / l.chunk : 0;
  if (l.nchunks > l.chunk_cap) {
    cudaFree(l.chunk_first);
    l.chunk_first = nullptr;
    l.chunk_cap = 0;
    TUNA_CUDA(pl, dev_alloc(&l.chunk_first, l.nchunks + 1));
    l.chunk_cap = l.nchunks;
  }
  if (l.nchunks > 0 && batch) {
    if (batch->n == kChunkBatch) {
      const int rc = launch_chunk_batch(pl, *batch, st);
      if (rc) return rc;
    }
    batch->b.it[batch->n++] = TunaChunkItem{l.pos, l.chunk_first, l.n, l.chunk, l.nchunks, l.total};
    batch->max_chunks = std::max(batch->max_chunks, l.nchunks);
  } else if (l.nchunks > 0) {
    const int th = 128;
    tuna_chunk_index_kernel<<<(unsigned)((l.nchunks + th) / th), th, 0, st>>>(
        l.pos, l.n, l.chunk, l.nchunks, l.total, l.chunk_first);
    TUNA_LAUNCHED(pl);
  }
  return TUNA_OK;
}

// scan of one list: per-rank warp scans, segment bases, (optionally) add bases
int scan_list(tuna_plan *pl, TunaList &l, int64_t seglen, int64_t nseg, int list_id,
              int64_t *wbase_slot, int uses_work, bool add_base, cudaStream_t st, int slot = 0) {
  int64_t *seg_total = pl->d_seg_total + (int64_t)slot * pl->topo.P;
  int64_t *seg_base = pl->d_seg_base + (int64_t)slot * pl->topo.P;
  if (seglen == 1 && add_base && l.kind == TUNA_LIST_DELIVER && l.n == nseg && nseg > 0) {
    // one block per segment (the self blocks): the positions are one scan of the spaced lengths
    tuna_segbase_kernel<<<1, 1024, 0, st>>>(l.len, nullptr, l.pos, nseg, pl->d_scal + 2 * list_id, wbase_slot,
                                            uses_work, l.pos + l.n, 1);
    TUNA_LAUNCHED(pl);
    return TUNA_OK;
  }
  if (nseg > 0 && seglen > 0) {
    const int th = 256;
    const int64_t blocks = (nseg * 32 + th - 1) / th;
    if (l.kind == TUNA_LIST_KEEP)
      tuna_segscan_kernel<1><<<(unsigned)blocks, th, 0, st>>>(l.len, l.pos, seg_total, pl->d_seg_raw,
                                                               seglen, nseg);
    else
      tuna_segscan_kernel<2><<<(unsigned)blocks, th, 0, st>>>(l.len, l.pos, seg_total, pl->d_seg_raw,
                                                               seglen, nseg);
    TUNA_LAUNCHED(pl);
  }
  tuna_segbase_kernel<<<1, 1024, 0, st>>>(seg_total, pl->d_seg_raw, seg_base,
                                          (nseg > 0 && seglen > 0) ? nseg : 0,
                                          pl->d_scal + 2 * list_id, wbase_slot, uses_work,
                                          l.pos + l.n, 0);
  TUNA_LAUNCHED(pl);
  if (add_base && l.n > 0) {
    const int th = 256;
    tuna_add_base_kernel<<<(unsigned)((l.n + th - 1) / th), th, 0, st>>>(l.pos, seg_base, seglen, l.n);
    TUNA_LAUNCHED(pl);
  }
  return TUNA_OK;
}

// The KEEP and the DELIVER list of a digit phase, scanned together: two launches
// instead of four.
int scan_phase_lists(tuna_plan *pl, TunaList &k, int64_t keep_seglen, int keep_id, int64_t *wbase_slot,
                     TunaList &d, int64_t del_seglen, int del_id, cudaStream_t st) {
  const int P = pl->topo.P;
  TunaScanArgs a{k.len, k.pos, pl->d_seg_total, pl->d_seg_raw, pl->d_seg_base, keep_seglen, P,
                 pl->d_scal + 2 * keep_id, wbase_slot, 1, k.pos + k.n};
  TunaScanArgs b{d.len, d.pos, pl->d_seg_total + P, pl->d_seg_raw + P, pl->d_seg_base + P, del_seglen, P,
                 pl->d_scal + 2 * del_id, nullptr, 0, d.pos + d.n};
  const int th = 256;
  const unsigned gx = (unsigned)(((int64_t)P * 32 + th - 1) / th);
  if (keep_seglen > 0 && del_seglen > 0) {
    tuna_segscan_pair_kernel<<<dim3(gx, 2), th, 0, st>>>(a, b);
    TUNA_LAUNCHED(pl);
  } else if (keep_seglen > 0) {  // (a phase with one list only runs the leaner single-list kernel)
    tuna_segscan_kernel<1><<<gx, th, 0, st>>>(a.val, a.out, a.seg_total, a.seg_raw, a.seglen, a.nseg);
    TUNA_LAUNCHED(pl);
  } else if (del_seglen > 0) {
    tuna_segscan_kernel<2><<<gx, th, 0, st>>>(b.val, b.out, b.seg_total, b.seg_raw, b.seglen, b.nseg);
    TUNA_LAUNCHED(pl);
  }
  tuna_segbase_pair_kernel<<<2, 1024, 0, st>>>(a, b);
  TUNA_LAUNCHED(pl);
  return TUNA_OK;
}

int validate_layout(int P, const int64_t *counts, const int64_t *sdispls, const int64_t *rdispls,
                    const int64_t *sendbase, const int64_t *recvbase) {
  if (!counts) return TUNA_ERR_INVALID_ARG;
  const int64_t PP = (int64_t)P * P;
  for (int64_t i = 0; i < PP; i++) {
    if (counts[i] < 0) return TUNA_ERR_INVALID_ARG;
    if (sdispls && sdispls[i] < 0) return TUNA_ERR_INVALID_ARG;
    if (rdispls && rdispls[i] < 0) return TUNA_ERR_INVALID_ARG;
  }
  for (int p = 0; p < P; p++) {
    if (sendbase && sendbase[p] < 0) return TUNA_ERR_INVALID_ARG;
    if (recvbase && recvbase[p] < 0) return TUNA_ERR_INVALID_ARG;
  }
  return TUNA_OK;
}

// What the host works out from a layout before anything touches the GPU.
struct HostLayout {
  std::vector<int64_t> sendbase, recvbase;  // elements
  int64_t payload = 0, send_extent = 0, recv_extent = 0;  // elements
};

// A few parked host threads for the pass over large count matrices (starting
// threads anew costs more than the pass itself).  One job at a time; created on
// first use and never torn down.
class HostPool {
 public:
  static HostPool &get() {
    static HostPool *pool = new HostPool();
    return *pool;
  }
  int size() const { return (int)workers_.size(); }
  bool usable() const { return !workers_.empty() && owner_ == getpid(); }  // threads do not survive a fork
  // Runs fn(i) for i in [0, n) on n of the parked threads and returns at once.
  void start(int n, std::function<void(int)> fn) {
    busy_.lock();
    std::lock_guard<std::mutex> lk(m_);
    job_ = std::move(fn);
    want_ = n;
    pending_ = n;
    gen_++;
    work_.notify_all();
  }
  void wait() {
    {
      std::unique_lock<std::mutex> lk(m_);
      done_.wait(lk, [&] { return pending_ == 0; });
    }
    busy_.unlock();
  }

 private:
  HostPool() : owner_(getpid()) {
    const unsigned hc = std::thread::hardware_concurrency();
    const int n = (int)std::min<unsigned>(8, hc > 1 ? hc - 1 : 0);
    for (int i = 0; i < n; i++) {
      workers_.emplace_back([this, i] { loop(i); });
      workers_.back().detach();
    }
  }
  void loop(int i) {
    unsigned seen = 0;
    for (;;) {
      std::unique_lock<std::mutex> lk(m_);
      work_.wait(lk, [&] { return gen_ != seen; });
      seen = gen_;
      if (i >= want_) continue;
      std::function<void(int)> f = job_;
      lk.unlock();
      f(i);
      lk.lock();
      if (--pending_ == 0) done_.notify_all();
    }
  }
  std::mutex m_, busy_;
  std::condition_variable work_, done_;
  std::function<void(int)> job_;
  std::vector<std::thread> workers_;
  unsigned gen_ = 0;
  int want_ = 0, pending_ = 0;
  pid_t owner_;
};

// Where the validated counts go on the device while the host's pass is still
// running (optional).
struct CountUpload {
  int64_t *d_dst = nullptr;
  cudaStream_t st = nullptr;
  bool done = false;       // out: every row has been handed to the copy engine
  cudaError_t err = cudaSuccess;
};

// The host's pass over the P x P matrices: rejects negative entries, sums the
// payload, finds every rank's region size and (copy_to) keeps a copy of the counts.
// Rows are walked in order, in blocks of rows that a few threads take in turn;
// rdispls, which is indexed [dst][src] against the counts' [src][dst], gets a
// second, tiled walk (64 x 64) so that both stay in cache.  With `up`, the calling
// thread sends every finished block of the copy to the device at once, in order,
// so the upload runs beside the pass instead of after it.
int host_layout(int P, const int64_t *counts, const int64_t *sdispls, const int64_t *rdispls,
                const int64_t *sendbase, const int64_t *recvbase, HostLayout *out,
                int64_t *copy_to = nullptr, CountUpload *up = nullptr) {
  if (!counts) return TUNA_ERR_INVALID_ARG;
  const int64_t PP = (int64_t)P * P;
  int nt = 1;
  HostPool *pool = nullptr;
  if (PP >= (1 << 20)) {
    pool = &HostPool::get();
    nt = pool->usable() ? pool->size() : 1;
    nt = (int)std::min<int64_t>(nt, env_i64("TUNA_HOST_THREADS", nt));
    nt = std::max(1, std::min(nt, P / 64));
  }
  const int nblk = nt == 1 ? 1 : 4 * nt;  // blocks of rows; thread t takes t, t + nt, ...
  auto row_of = [&](int k) { return (int)((int64_t)P * k / nblk); };
  std::vector<int64_t> sreg(P, 0);
  std::vector<std::vector<int64_t>> rpart(nt, std::vector<int64_t>(P, 0));
  std::vector<int64_t> pay(nt, 0);
  std::vector<char> badv(nt, 0);
  std::vector<std::atomic<int>> ready(nblk);
  for (auto &r : ready) r.store(0, std::memory_order_relaxed);
  auto work = [&](int t) {
    int64_t payload = 0;
    bool bad = false;
    int64_t *rr = rpart[t].data();
    for (int k = t; k < nblk; k += nt) {
      const int s_lo = row_of(k), s_hi = row_of(k + 1);
      for (int s = s_lo; s < s_hi; s++) {
        const int64_t *crow = counts + (int64_t)s * P;
        const int64_t *drow = sdispls ? sdispls + (int64_t)s * P : nullptr;
        int64_t *keep = copy_to ? copy_to + (int64_t)s * P : nullptr;
        int64_t sr = 0;
        for (int d = 0; d < P; d++) {
          const int64_t c = crow[d];
          if (keep) keep[d] = c;
          bad |= c < 0;
          payload += c;
          if (drow) {
            bad |= drow[d] < 0;
            sr = std::max(sr, drow[d] + c);
          } else {
            sr += c;
          }
          if (!rdispls) rr[d] += c;
        }
        sreg[s] = sr;
      }
      ready[k].store(1, std::memory_order_release);  // the copy of these rows is complete
      if (rdispls) {
        constexpr int T = 64;
        for (int s0 = s_lo; s0 < s_hi; s0 += T)
          for (int d0 = 0; d0 < P; d0 += T) {
            const int s1 = std::min(s_hi, s0 + T), d1 = std::min(P, d0 + T);
            for (int d = d0; d < d1; d++) {
              const int64_t *xrow = rdispls + (int64_t)d * P;
              int64_t m = rr[d];
              for (int s = s0; s < s1; s++) {
                const int64_t x = xrow[s];
                bad |= x < 0;
                m = std::max(m, x + counts[(int64_t)s * P + d]);
              }
              rr[d] = m;
            }
          }
      }
    }
    pay[t] = payload;
    badv[t] = bad;
  };
  auto send_block = [&](int k) {  // rows of block k: host copy -> device
    const int64_t lo = (int64_t)row_of(k) * P, hi = (int64_t)row_of(k + 1) * P;
    if (hi > lo && up->err == cudaSuccess)
      up->err = cudaMemcpyAsync(up->d_dst + lo, copy_to + lo, (size_t)(hi - lo) * 8, cudaMemcpyHostToDevice, up->st);
  };
  const bool streaming = up && copy_to && nt > 1;
  if (nt == 1) {
    work(0);
  } else {
    pool->start(nt, work);
    if (streaming)
      for (int k = 0; k < nblk; k++) {
        while (ready[k].load(std::memory_order_acquire) == 0) std::this_thread::yield();
        send_block(k);
      }
    pool->wait();
  }
  if (streaming) {
    if (up->err != cudaSuccess) return TUNA_ERR_CUDA;
    up->done = true;
  }
  bool bad = false;
  int64_t payload = 0;
  std::vector<int64_t> rreg(P, 0);
  for (int t = 0; t < nt; t++) {
    bad |= badv[t] != 0;
    payload += pay[t];
    for (int d = 0; d < P; d++) rreg[d] = rdispls ? std::max(rreg[d], rpart[t][d]) : rreg[d] + rpart[t][d];
  }
  for (int p = 0; p < P; p++) bad |= (sendbase && sendbase[p] < 0) || (recvbase && recvbase[p] < 0);
  if (bad) return TUNA_ERR_INVALID_ARG;
  out->sendbase.resize(P);
  out->recvbase.resize(P);
  int64_t se = 0, re = 0, acc_s = 0, acc_r = 0;
  for (int p = 0; p < P; p++) {
    out->sendbase[p] = sendbase ? sendbase[p] : acc_s;
    out->recvbase[p] = recvbase ? recvbase[p] : acc_r;
    acc_s += sreg[p];
    acc_r += rreg[p];
    se = std::max(se, out->sendbase[p] + sreg[p]);
    re = std::max(re, out->recvbase[p] + rreg[p]);
  }
  out->payload = payload;
  out->send_extent = se;
  out->recv_extent = re;
  return TUNA_OK;
}

// Updates from device counts enqueue the same kernels with the same arguments every
// time (the plan's tables never move), a few dozen short launches: they are captured
// once, on a stream of the plan's own, and replayed as one graph launch on the
// caller's stream.  TUNA_PLAN_GRAPH=0 turns this off; so does any failure to capture.
template <class F>
int replay_tables_graph(tuna_plan *pl, F &enqueue, cudaStream_t st) {
  static const bool enabled = env_i64("TUNA_PLAN_GRAPH", 1) != 0;
  if (!enabled) return enqueue(st);
  if (pl->tables_graph && pl->tables_graph_counts != pl->d_counts) {
    cudaGraphExecDestroy(pl->tables_graph);
    pl->tables_graph = nullptr;
  }
  if (!pl->tables_graph) {
    if (!pl->capture_stream &&
        cudaStreamCreateWithFlags(&pl->capture_stream, cudaStreamNonBlocking) != cudaSuccess) {
      (void)cudaGetLastError();
      pl->capture_stream = nullptr;
      return enqueue(st);
    }
    if (cudaStreamBeginCapture(pl->capture_stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
      (void)cudaGetLastError();
      return enqueue(st);
    }
    const int64_t before = pl->launch_count;
    const int rc = enqueue(pl->capture_stream);
    cudaGraph_t g = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(pl->capture_stream, &g);
    pl->tables_graph_launches = pl->launch_count - before;
    pl->launch_count = before;  // nothing has run yet
    cudaGraphExec_t ex = nullptr;
    if (rc == TUNA_OK && ce == cudaSuccess && g && cudaGraphInstantiate(&ex, g, 0) == cudaSuccess) {
      pl->tables_graph = ex;
      pl->tables_graph_counts = pl->d_counts;
    }
    if (g) cudaGraphDestroy(g);
    if (!pl->tables_graph) {
      (void)cudaGetLastError();
      pl->cuda_err = 0;
      return enqueue(st);
    }
  }
  TUNA_CUDA(pl, cudaGraphLaunch(pl->tables_graph, st));
  pl->launch_count += pl->tables_graph_launches;
  return TUNA_OK;
}

// Uploads the layout, runs every plan kernel, reads the totals back.  Without a
// host layout (`hl` null) the counts are already in pl->d_counts and the layout
// is packed: region bases, extents and the payload are worked out on the device.
int build_tables(tuna_plan *pl, const HostLayout *hl, const int64_t *sdispls, const int64_t *rdispls,
                 cudaStream_t st) {
  const int64_t *counts = pl->h_counts;  // validated and copied by host_layout
  const TunaTopo &t = pl->topo;
  const int P = t.P;
  const int64_t PP = (int64_t)P * P;
  int rc = TUNA_OK;

  rc = wait_in_flight(pl);  // an exchange that is still running reads the tables rewritten below
  if (rc) return rc;
  pl->rows_valid = false;  // a row list belongs to the counts it was built for
  pl->tables_valid = false;
  // host copies for the checks at call time
  pl->have_sdispls = sdispls != nullptr;
  pl->have_rdispls = rdispls != nullptr;
  if (sdispls) pl->h_sdispls.assign(sdispls, sdispls + PP); else pl->h_sdispls.clear();
  if (rdispls) pl->h_rdispls.assign(rdispls, rdispls + PP); else pl->h_rdispls.clear();
  pl->h_counts_valid = hl != nullptr;

  const int th = 256;
  const unsigned gPP = (unsigned)((PP + th - 1) / th);
  const unsigned gseg = (unsigned)(((int64_t)P * 32 + th - 1) / th);
  const int nph = (int)pl->phases.size();
  const int nlists = 2 * nph + 2;
  // Everything from the layout to the self-check only enqueues work on one stream
  // and reads nothing back, so it can run directly or be captured as a graph.
  auto enqueue_tables = [&](cudaStream_t st) -> int {
    int rc = TUNA_OK;
    // list totals, workspace offsets, extents, per-round bytes and self-check counters
    // all start from zero: they are slices of one block
    TUNA_CUDA(pl, cudaMemsetAsync(pl->d_readback, 0, (size_t)pl->readback_words * 8, st));
    if (hl) {
      pl->payload = hl->payload * t.elem;
      pl->send_extent = hl->send_extent * t.elem;
      pl->recv_extent = hl->recv_extent * t.elem;
      if (!pl->counts_uploaded)
        TUNA_CUDA(pl, cudaMemcpyAsync(pl->d_counts, counts, PP * 8, cudaMemcpyHostToDevice, st));
      TUNA_CUDA(pl, cudaMemcpyAsync(pl->d_sendbase, hl->sendbase.data(), P * 8, cudaMemcpyHostToDevice, st));
      TUNA_CUDA(pl, cudaMemcpyAsync(pl->d_recvbase, hl->recvbase.data(), P * 8, cudaMemcpyHostToDevice, st));
      const int64_t ext[4] = {pl->send_extent, pl->recv_extent, hl->payload, 0};
      TUNA_CUDA(pl, cudaMemcpyAsync(pl->d_extents, ext, sizeof(ext), cudaMemcpyHostToDevice, st));
      // (pageable sources: the runtime stages these copies before it returns)
    }
    pl->counts_uploaded = false;
    if (sdispls) {
      TUNA_CUDA(pl, cudaMemcpyAsync(pl->d_sdispls, sdispls, PP * 8, cudaMemcpyHostToDevice, st));
    } else {  // packed: exclusive scan of every rank's row of counts
      tuna_segscan_kernel<0><<<gseg, th, 0, st>>>(pl->d_counts, pl->d_sdispls, pl->d_seg_total,
                                                   nullptr, P, P);
      TUNA_LAUNCHED(pl);
      if (!hl) {  // send regions laid end to end: bases = scan of the row sums
        tuna_segbase_kernel<<<1, 1024, 0, st>>>(pl->d_seg_total, nullptr, pl->d_sendbase, P, pl->d_scal, nullptr, 0,
                                                nullptr, 0);
        TUNA_LAUNCHED(pl);
        tuna_packed_extents_kernel<<<1, 32, 0, st>>>(pl->d_scal, t.elem, pl->d_extents);
        TUNA_LAUNCHED(pl);
      }
    }
    if (rdispls) {
      TUNA_CUDA(pl, cudaMemcpyAsync(pl->d_rdispls, rdispls, PP * 8, cudaMemcpyHostToDevice, st));
    } else {  // packed: scan of the receive counts = rows of the transposed matrix
      tuna_transpose_kernel<<<dim3((P + 31) / 32, (P + 31) / 32), dim3(32, 8), 0, st>>>(pl->d_counts, pl->d_tmp, P, hl ? nullptr : pl->d_extents + 3);
      TUNA_LAUNCHED(pl);
      tuna_segscan_kernel<0><<<gseg, th, 0, st>>>(pl->d_tmp, pl->d_rdispls, pl->d_seg_total,
                                                   nullptr, P, P);
      TUNA_LAUNCHED(pl);
      if (!hl) {  // receive regions likewise: scan of the column sums
        tuna_segbase_kernel<<<1, 1024, 0, st>>>(pl->d_seg_total, nullptr, pl->d_recvbase, P, pl->d_scal, nullptr, 0,
                                                nullptr, 0);
        TUNA_LAUNCHED(pl);
      }
    }

    if (pl->classic) {
      TUNA_CUDA(pl, cudaMemsetAsync(pl->rot.len, 0, (size_t)PP * 8, st));
      TUNA_CUDA(pl, cudaMemsetAsync(pl->rot.src, 0, (size_t)PP * 8, st));
      TUNA_CUDA(pl, cudaMemsetAsync(pl->rot.dst, 0, (size_t)PP * 8, st));
    }
    tuna_init_tables_kernel<<<gPP, th, 0, st>>>(t, pl->d_counts, pl->d_sdispls, pl->d_rdispls,
                                                pl->d_sendbase, pl->d_recvbase, pl->d_sz[0],
                                                pl->d_loc[0], pl->dir.len, pl->dir.src, pl->dir.dst,
                                                pl->rot.len, pl->rot.src, pl->rot.dst,
                                                pl->classic ? 1 : 0);
    TUNA_LAUNCHED(pl);

    int cur = 0;
    for (int f = 0; f < nph; f++) {
      const TunaPhase &ph = pl->phases[f];
      TunaList &k = pl->keep[f];
      TunaList &d = pl->deliver[f];
      if (ph.stag_hi > 0) {  // a batch of the staggered exchange: every block arrives
        const int64_t nd = (int64_t)P * (ph.stag_hi - ph.stag_lo);
        tuna_stagger_batch_kernel<<<(unsigned)((nd + th - 1) / th), th, 0, st>>>(
            t, ph.stag_lo, ph.stag_hi, pl->d_sz[cur], pl->d_loc[cur], pl->d_rdispls, pl->d_recvbase,
            d.len, d.src, d.dst, pl->d_round_bytes + ph.stats_off);
        TUNA_LAUNCHED(pl);
        rc = scan_list(pl, k, 0, P, f, pl->d_wbase + f, 1, false, st, 0);
        if (rc) return rc;
        rc = scan_list(pl, d, ph.finals, P, nph + f, nullptr, 0, true, st, 1);
        if (rc) return rc;
        continue;
      }
      PhaseDev pd{ph.level, ph.radix, ph.count, ph.stride, ph.moving, ph.per_rank, ph.finals};
      if (ph.level == 0 && ph.stride == 1 && ph.radix >= t.Q && t.N <= 65535) {
        const unsigned tiles = (unsigned)((t.Q + 31) / 32);
        tuna_meta_exchange_diag_kernel<<<dim3(tiles * tiles, t.N, t.N), dim3(32, 8), 0, st>>>(
            t, pd, pl->d_sz[cur], pl->d_loc[cur], pl->d_sz[cur ^ 1], k.len, k.src, d.len, d.src,
            pl->d_round_bytes + ph.stats_off);
      } else {
        const size_t smem = ph.radix <= 4096 ? (size_t)ph.radix * 8 : 0;
        tuna_meta_exchange_kernel<<<gPP, th, smem, st>>>(t, pd, pl->d_sz[cur], pl->d_loc[cur],
                                                         pl->d_sz[cur ^ 1], k.len, k.src, d.len, d.src,
                                                         pl->d_round_bytes + ph.stats_off);
      }
      TUNA_LAUNCHED(pl);
      // per-rank prefix sums of both lists; the KEEP stream is this phase's workspace region
      rc = scan_phase_lists(pl, k, ph.per_rank - ph.finals, f, pl->d_wbase + f, d, ph.finals, nph + f, st);
      if (rc) return rc;
      tuna_place_kernel<<<gPP, th, 0, st>>>(t, pd, pl->d_loc[cur], pl->d_loc[cur ^ 1], k.pos,
                                            pl->d_seg_base, k.len, d.pos, pl->d_seg_base + P, d.dst,
                                            pl->d_wbase + f, pl->d_rdispls, pl->d_recvbase,
                                            pl->classic ? 1 : 0, pl->rot.len, pl->rot.src, pl->rot.dst);
      TUNA_LAUNCHED(pl);
      cur ^= 1;
    }
    // work partitions of the rotation and direct lists
    rc = scan_list(pl, pl->rot, pl->classic ? P : 1, P, 2 * nph, nullptr, 0, true, st);
    if (rc) return rc;
    if (!pl->dir_shared && !pl->no_direct) rc = scan_list(pl, pl->dir, P, P, 2 * nph + 1, nullptr, 0, true, st);
    if (rc) return rc;

    // self-check: every descriptor of every list stays inside its buffers
    // (the same pass sums, per list, the bytes of the blocks whose source and
    // destination differ modulo 16: they pick the kernel build)
    if (pl->n_check_items > 0) {
      const unsigned gx = (unsigned)std::min<int64_t>((pl->check_max_n + th - 1) / th, 148 * 8);
      tuna_check_lists_kernel<<<dim3(gx, pl->n_check_items), th, 0, st>>>(
          static_cast<const TunaCheckItem *>(pl->d_check_items), pl->d_extents, pl->d_wbase + nph, pl->d_wbase,
          pl->d_violations);
      TUNA_LAUNCHED(pl);
    }

    return rc;
  };
  Timed plan_timer(pl, TUNA_TIMER_PLAN, 0, st);
  rc = hl ? enqueue_tables(st) : replay_tables_graph(pl, enqueue_tables, st);
  if (rc) return rc;
  plan_timer.stop();  // the chunk tables below are timed separately, after the read-back
  // one read-back: stream totals, workspace offsets, per-round bytes
  std::vector<int64_t> scal(2 * (2 * nph + 2)), wbase(nph + 1);
  std::vector<unsigned long long> rbytes(std::max<int64_t>(pl->stats_n, 1));
  std::vector<unsigned long long> checked(1 + nlists);
  int64_t ext[4] = {0, 0, 0, 0};
  if (pl->h_readback) {  // one copy of the whole block into pinned memory
    TUNA_CUDA(pl, cudaMemcpyAsync(pl->h_readback, pl->d_readback, (size_t)pl->readback_words * 8,
                                  cudaMemcpyDeviceToHost, st));
    TUNA_CUDA(pl, cudaStreamSynchronize(st));
    const int64_t *h = pl->h_readback;
    std::copy(h + (pl->d_scal - pl->d_readback), h + (pl->d_scal - pl->d_readback) + scal.size(), scal.begin());
    std::copy(h + (pl->d_wbase - pl->d_readback), h + (pl->d_wbase - pl->d_readback) + wbase.size(), wbase.begin());
    std::copy(h + (pl->d_extents - pl->d_readback), h + (pl->d_extents - pl->d_readback) + 4, ext);
    const unsigned long long *hu = reinterpret_cast<const unsigned long long *>(h);
    const int64_t o_rb = reinterpret_cast<int64_t *>(pl->d_round_bytes) - pl->d_readback;
    const int64_t o_vi = reinterpret_cast<int64_t *>(pl->d_violations) - pl->d_readback;
    std::copy(hu + o_rb, hu + o_rb + rbytes.size(), rbytes.begin());
    std::copy(hu + o_vi, hu + o_vi + checked.size(), checked.begin());
  } else {
    TUNA_CUDA(pl, cudaMemcpyAsync(scal.data(), pl->d_scal, scal.size() * 8, cudaMemcpyDeviceToHost, st));
    TUNA_CUDA(pl, cudaMemcpyAsync(wbase.data(), pl->d_wbase, wbase.size() * 8, cudaMemcpyDeviceToHost, st));
    TUNA_CUDA(pl, cudaMemcpyAsync(rbytes.data(), pl->d_round_bytes, rbytes.size() * 8,
                                  cudaMemcpyDeviceToHost, st));
    TUNA_CUDA(pl, cudaMemcpyAsync(checked.data(), pl->d_violations, checked.size() * 8, cudaMemcpyDeviceToHost, st));
    TUNA_CUDA(pl, cudaMemcpyAsync(ext, pl->d_extents, sizeof(ext), cudaMemcpyDeviceToHost, st));
    TUNA_CUDA(pl, cudaStreamSynchronize(st));
  }
  if (!hl) {
    if (ext[3] != 0) return TUNA_ERR_INVALID_ARG;  // negative counts
    pl->send_extent = ext[0];
    pl->recv_extent = ext[1];
    pl->payload = ext[2] * t.elem;
  }
  if (checked[0] != 0) return TUNA_ERR_INTERNAL;
  pl->h_wbase = wbase;
  auto take = [&](TunaList &l, int id) {
    l.total = scal[2 * id];
    l.bytes = scal[2 * id + 1];
    l.unaligned_bytes = (int64_t)checked[1 + id];
  };
  for (int f = 0; f < nph; f++) {
    take(pl->keep[f], f);
    take(pl->deliver[f], nph + f);
  }
  take(pl->rot, 2 * nph);
  if (!pl->dir_shared && !pl->no_direct) take(pl->dir, 2 * nph + 1);
  pl->workspace_need = wbase[nph];
  for (auto &r : pl->rounds) r.bytes = (int64_t)rbytes[r.stat];

  Timed chunk_timer(pl, TUNA_TIMER_PLAN, 0, st);
  ChunkCollector cc;  // the chunk tables of all lists: one launch (per 32 lists)
  for (int f = 0; f < nph; f++) {
    rc = build_chunks(pl, pl->keep[f], st, &cc);
    if (rc) return rc;
    rc = build_chunks(pl, pl->deliver[f], st, &cc);
    if (rc) return rc;
  }
  rc = build_chunks(pl, pl->rot, st, &cc);
  if (rc) return rc;
  if (!pl->dir_shared && !pl->no_direct) rc = build_chunks(pl, pl->dir, st, &cc);
  if (rc) return rc;
  rc = launch_chunk_batch(pl, cc, st);
  if (rc) return rc;
  rc = mark_tables_ready(pl, st);  // (no second wait on the host: exchanges order themselves behind this)
  if (rc) return rc;
  pl->tables_valid = true;
  return TUNA_OK;
}

void add_level(tuna_plan *pl, int level, int count, int radix, int other) {
  const int w = num_digits(count, radix);
  for (int x = 0; x < w; x++) {
    TunaPhase ph{};
    ph.level = level;
    ph.x = x;
    ph.radix = radix;
    ph.count = count;
    ph.stride = ipow64(radix, x);
    ph.moving = count - count_digit(count, radix, x, 0);
    ph.per_rank = ph.moving * other;
    // blocks whose higher digits are all zero arrive in this phase: the offsets
    // below radix^(x+1) with a non-zero digit x (own group only, for local phases)
    const int64_t arrive = std::min<int64_t>(count, ph.stride * radix) - std::min<int64_t>(count, ph.stride);
    ph.finals = pl->classic ? 0 : (level == 0 ? arrive : arrive * other);
    ph.stats_off = pl->stats_n;
    pl->stats_n += radix;
    const int phase = (int)pl->phases.size();
    pl->phases.push_back(ph);
    for (int z = 1; z < radix; z++) {
      if ((int64_t)z * ph.stride >= count) continue;
      tuna_plan::Round r{};
      r.level = level;
      r.x = x;
      r.z = z;
      r.phase = phase;
      r.stat = ph.stats_off + z;
      // level 0 counts blocks, level 1 super-blocks (Q blocks each)
      r.units = (int64_t)pl->topo.P * count_digit(count, radix, x, z) * (level == 0 ? other : 1);
      pl->rounds.push_back(r);
    }
  }
}

// Staggered inter-group exchange (Algorithm 2): the step index ii = gi*Q + gr runs
// over [0, P) in batches of block_count; the first Q indices (gi = 0) name the own
// group and move nothing.  Every batch that moves something becomes one launch.
void add_staggered(tuna_plan *pl, int block_count) {
  const int P = pl->topo.P, Q = pl->topo.Q, N = pl->topo.N;
  const int64_t stats_off = pl->stats_n;
  pl->stats_n += P;
  int batch = 0;
  for (int64_t lo0 = 0; lo0 < P; lo0 += block_count) {
    const int lo = (int)std::max<int64_t>(lo0, Q), hi = (int)std::min<int64_t>(P, lo0 + block_count);
    if (hi <= lo) continue;
    TunaPhase ph{};
    ph.level = 1;
    ph.x = batch++;
    ph.radix = N;
    ph.count = N;
    ph.stride = 1;
    ph.moving = ph.per_rank = ph.finals = hi - lo;
    ph.stats_off = stats_off;
    ph.stag_lo = lo;
    ph.stag_hi = hi;
    const int phase = (int)pl->phases.size();
    pl->phases.push_back(ph);
    for (int ii = lo; ii < hi; ii++) {
      tuna_plan::Round r{};
      r.level = 1;
      r.x = ii / Q;  // gi
      r.z = ii % Q;  // gr
      r.phase = phase;
      r.stat = stats_off + ii;
      r.units = P;   // one block per rank
      pl->rounds.push_back(r);
    }
  }
}

int check_call_args(tuna_plan *pl, const int64_t *sendcounts, const int64_t *sdispls,
                    const int64_t *recvcounts, const int64_t *rdispls) {
  const int P = pl->topo.P;
  const int64_t PP = (int64_t)P * P;
  if (!pl->tables_valid) return TUNA_ERR_INTERNAL;  // the last update failed: the plan must not be used
  if (!pl->h_counts_valid && (sendcounts || sdispls || recvcounts || rdispls)) {
    // the counts came from device memory: fetch them for the comparison, once
    TUNA_CUDA(pl, cudaMemcpy(pl->h_buf[pl->h_cur], pl->d_counts, (size_t)PP * 8, cudaMemcpyDeviceToHost));
    pl->h_counts = pl->h_buf[pl->h_cur];
    pl->h_counts_valid = true;
  }
  if (sendcounts && memcmp(sendcounts, pl->h_counts, PP * 8) != 0) return TUNA_ERR_COUNT_MISMATCH;
  if (recvcounts)
    for (int d = 0; d < P; d++)
      for (int s = 0; s < P; s++)
        if (recvcounts[(int64_t)d * P + s] != pl->h_counts[(int64_t)s * P + d])
          return TUNA_ERR_COUNT_MISMATCH;
  if (sdispls) {
    if (pl->have_sdispls) {
      if (memcmp(sdispls, pl->h_sdispls.data(), PP * 8) != 0) return TUNA_ERR_COUNT_MISMATCH;
    } else {
      for (int s = 0; s < P; s++) {
        int64_t acc = 0;
        for (int d = 0; d < P; d++) {
          if (sdispls[(int64_t)s * P + d] != acc) return TUNA_ERR_COUNT_MISMATCH;
          acc += pl->h_counts[(int64_t)s * P + d];
        }
      }
    }
  }
  if (rdispls) {
    if (pl->have_rdispls) {
      if (memcmp(rdispls, pl->h_rdispls.data(), PP * 8) != 0) return TUNA_ERR_COUNT_MISMATCH;
    } else {
      for (int d = 0; d < P; d++) {
        int64_t acc = 0;
        for (int s = 0; s < P; s++) {
          if (rdispls[(int64_t)d * P + s] != acc) return TUNA_ERR_COUNT_MISMATCH;
          acc += pl->h_counts[(int64_t)s * P + d];
        }
      }
    }
  }
  return TUNA_OK;
}

bool ranges_overlap(const void *a, size_t na, const void *b, size_t nb) {
  const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
  return na > 0 && nb > 0 && a0 < b0 + nb && b0 < a0 + na;
}

TunaListArgs list_args(const TunaList &l) {
  TunaListArgs a{};
  a.len = l.len;
  a.pos = l.pos;
  a.src = l.src;
  a.dst = l.dst;
  a.chunk_first = l.chunk_first;
  a.n = l.n;
  a.total = l.total;
  a.chunk = l.chunk;
  a.nchunks = l.n > 0 ? l.nchunks : 0;
  return a;
}

TunaMoveArgs move_args(const tuna_plan *pl, const void *send, void *recv, char *work) {
  TunaMoveArgs a{};
  a.base[TUNA_BUF_SEND] = (char *)const_cast<void *>(send);
  a.base[TUNA_BUF_RECV] = (char *)recv;
  a.base[TUNA_BUF_WORK] = work;
  a.extent[TUNA_BUF_SEND] = pl->send_extent;
  a.extent[TUNA_BUF_RECV] = pl->recv_extent;
  a.extent[TUNA_BUF_WORK] = work ? pl->workspace_need : 0;
  a.keep_base = 0;
  a.error = pl->d_error;
  a.bulk_off = (pl->flags & TUNA_FLAG_BULK_COPY) ? 1 : 0;
  return a;
}

// One launch per digit phase: its KEEP list, its DELIVER list and, riding along in
// the first launch, the self blocks (they depend on nothing).  In classic mode
// the rotation list needs every phase finished and gets a launch of its own.
int run_tuna(tuna_plan *pl, const void *send, void *recv, cudaStream_t st) {
  {
    const int arc = await_tables(pl, st);
    if (arc) return arc;
  }
  if (pl->workspace_need > 0 &&
      (!pl->workspace || pl->workspace_bytes < (size_t)pl->workspace_need))
    return TUNA_ERR_WORKSPACE;
  int launches = 0;
  bool rot_done = pl->rot.nchunks == 0;
  for (size_t f = 0; f < pl->phases.size(); f++) {
    const int kind = pl->phases[f].level == 0 ? TUNA_TIMER_ROUND_LOCAL : TUNA_TIMER_ROUND_GLOBAL;
    const TunaList &k = pl->keep[f];
    const TunaList &d = pl->deliver[f];
    const bool with_rot = !rot_done && !pl->classic;
    if (k.nchunks == 0 && d.nchunks == 0 && !with_rot) continue;
    TunaMoveArgs a = move_args(pl, send, recv, pl->workspace);
    a.keep = list_args(k);
    a.del = list_args(d);
    a.keep_base = pl->h_wbase[f];
    int64_t bytes = k.bytes + d.bytes;
    // the lists of a launch share one kernel build: the one most of its bytes want
    int64_t small_bytes = (k.small_blocks ? k.bytes : 0) + (d.small_blocks ? d.bytes : 0);
    if (with_rot) {
      a.rot = list_args(pl->rot);
      bytes += pl->rot.bytes;
      small_bytes += pl->rot.small_blocks ? pl->rot.bytes : 0;
      rot_done = true;
    }
    const bool small = 2 * small_bytes >= bytes;
    Timed tm(pl, kind, bytes, st);
    TUNA_CUDA(pl, tuna_launch_move(TUNA_K_ROUND, a, small, st));
    launches++;
  }
  if (!rot_done) {
    Timed tm(pl, TUNA_TIMER_ROTATE, pl->rot.bytes, st);
    TunaMoveArgs a = move_args(pl, send, recv, pl->workspace);
    a.rot = list_args(pl->rot);
    TUNA_CUDA(pl, tuna_launch_move(TUNA_K_ROTATE, a, pl->rot.small_blocks, st));
    launches++;
  }
  pl->last_launches = launches;
  pl->launch_count += launches;
  return launches > 0 ? mark_in_flight(pl, st) : TUNA_OK;
}

int run_direct(tuna_plan *pl, const void *send, void *recv, cudaStream_t st) {
  if (pl->no_direct) return TUNA_ERR_INVALID_ARG;  // the plan was created without a direct list
  {
    const int arc = await_tables(pl, st);
    if (arc) return arc;
  }
  int launches = 0;
  if (pl->dir_shared) {  // the single phase's DELIVER list and the self blocks: every block, once
    const TunaList &d = pl->deliver[0];
    if (d.nchunks > 0 || pl->rot.nchunks > 0) {
      const int64_t bytes = d.bytes + pl->rot.bytes;
      const int64_t small_bytes = (d.small_blocks ? d.bytes : 0) + (pl->rot.small_blocks ? pl->rot.bytes : 0);
      Timed tm(pl, TUNA_TIMER_DIRECT, bytes, st);
      TunaMoveArgs a = move_args(pl, send, recv, nullptr);
      a.del = list_args(d);
      a.rot = list_args(pl->rot);
      TUNA_CUDA(pl, tuna_launch_move(TUNA_K_DIRECT, a, 2 * small_bytes >= bytes, st));
      launches++;
    }
  } else if (pl->dir.nchunks > 0) {
    Timed tm(pl, TUNA_TIMER_DIRECT, pl->dir.bytes, st);
    TunaMoveArgs a = move_args(pl, send, recv, nullptr);
    a.del = list_args(pl->dir);
    TUNA_CUDA(pl, tuna_launch_move(TUNA_K_DIRECT, a, pl->dir.small_blocks, st));
    launches++;
  }
  pl->last_launches = launches;
  pl->launch_count += launches;
  return launches > 0 ? mark_in_flight(pl, st) : TUNA_OK;
}

int64_t align256(int64_t v) { return (v + 255) & ~(int64_t)255; }

}  // namespace

// ------------------------------------------------------------------ C ABI

extern "C" {

int tuna_version(void) { return 100; }

const char *tuna_strerror(int status) {
  switch (status) {
    case TUNA_OK: return "success";
    case TUNA_ERR_INVALID_ARG: return "invalid argument";
    case TUNA_ERR_BAD_RADIX: return "radix out of range";
    case TUNA_ERR_BAD_HIERARCHY: return "l * g != P";
    case TUNA_ERR_COUNT_MISMATCH: return "counts or displacements do not match the plan";
    case TUNA_ERR_OVERLAP: return "send and receive buffers overlap";
    case TUNA_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case TUNA_ERR_CUDA: return "CUDA runtime error";
    case TUNA_ERR_NOMEM: return "out of memory";
    case TUNA_ERR_RANGE: return "index or size out of range";
    case TUNA_ERR_INTERNAL: return "the plan's self-check found a descriptor outside its buffers";
    default: return "unknown status";
  }
}

int tuna_plan_destroy(tuna_plan_t *pl) {
  if (!pl) return TUNA_OK;
  if (pl->in_flight) {
    if (pl->in_flight_set) (void)cudaEventSynchronize(pl->in_flight);  // the tables are freed below
    cudaEventDestroy(pl->in_flight);
  }
  if (pl->tables_ready) {
    if (pl->tables_ready_set) (void)cudaEventSynchronize(pl->tables_ready);
    cudaEventDestroy(pl->tables_ready);
  }
  if (pl->tables_graph) cudaGraphExecDestroy(pl->tables_graph);
  if (pl->capture_stream) cudaStreamDestroy(pl->capture_stream);
  for (auto &l : pl->keep) free_list(l);
  for (auto &l : pl->deliver) free_list(l);
  free_list(pl->rot);
  free_list(pl->dir);
  free_list(pl->rowsl);
  cudaFree(pl->d_row_start);
  for (int i = 0; i < 2; i++) {
    if (pl->h_pinned)
      cudaFreeHost(pl->h_buf[i]);
    else
      free(pl->h_buf[i]);
  }
  cudaFree(pl->d_counts_buf[0]);
  cudaFree(pl->d_counts_buf[1]);
  cudaFree(pl->d_sdispls);
  cudaFree(pl->d_rdispls);
  cudaFree(pl->d_sendbase);
  cudaFree(pl->d_recvbase);
  for (int i = 0; i < 2; i++) {
    cudaFree(pl->d_sz[i]);
    cudaFree(pl->d_loc[i]);
  }
  cudaFree(pl->d_seg_total);
  cudaFree(pl->d_seg_raw);
  cudaFree(pl->d_seg_base);
  cudaFree(pl->d_tmp);
  cudaFree(pl->d_check_items);
  cudaFree(pl->d_readback);  // (d_scal, d_wbase, d_extents, d_round_bytes, d_violations are slices of it)
  if (pl->h_readback) cudaFreeHost(pl->h_readback);
  cudaFree(pl->d_error);
  for (auto &s : pl->stamps) {
    cudaEventDestroy(s.a);
    cudaEventDestroy(s.b);
  }
  for (auto e : pl->event_pool) cudaEventDestroy(e);
  delete pl;
  return TUNA_OK;
}

static int plan_create(tuna_plan_t **out, int P, int radix, int radix_global, int block_count,
                       int l, int g, int elem_size, unsigned flags, const int64_t *sendcounts,
                       const int64_t *sdispls, const int64_t *rdispls, const int64_t *sendbase,
                       const int64_t *recvbase, void *stream) {
  if (!out) return TUNA_ERR_INVALID_ARG;
  *out = nullptr;
  if (P < 1 || P > 32768 || elem_size < 1 || !sendcounts || l < 1 || g < 1) return TUNA_ERR_INVALID_ARG;
  if ((int64_t)l * g != P) return TUNA_ERR_BAD_HIERARCHY;
  if (radix < 2 || radix > std::max(2, l)) return TUNA_ERR_BAD_RADIX;
  if (block_count == 0 && g > 1 && (radix_global < 2 || radix_global > std::max(2, g)))
    return TUNA_ERR_BAD_RADIX;
  if (block_count < 0 || (block_count > 0 && (flags & TUNA_FLAG_CLASSIC_ROTATE)))
    return TUNA_ERR_INVALID_ARG;
  tuna_plan *pl = new (std::nothrow) tuna_plan();
  if (!pl) return TUNA_ERR_NOMEM;
  // host buffers for the counts: pinned if possible (the upload then runs at the
  // host link's rate and without a staging copy), plain memory otherwise
  {
    const size_t bytes = (size_t)P * P * sizeof(int64_t);
    void *a = nullptr, *b = nullptr;
    if (cudaHostAlloc(&a, bytes, cudaHostAllocDefault) == cudaSuccess &&
        cudaHostAlloc(&b, bytes, cudaHostAllocDefault) == cudaSuccess) {
      pl->h_pinned = true;
    } else {
      (void)cudaGetLastError();
      if (a) cudaFreeHost(a);
      a = malloc(bytes);
      b = malloc(bytes);
    }
    pl->h_buf[0] = (int64_t *)a;
    pl->h_buf[1] = (int64_t *)b;
    if (!a || !b) {
      tuna_plan_destroy(pl);
      return TUNA_ERR_NOMEM;
    }
  }
  HostLayout hl;
  int rc = host_layout(P, sendcounts, sdispls, rdispls, sendbase, recvbase, &hl, pl->h_buf[0]);
  if (rc) {
    tuna_plan_destroy(pl);
    return rc;
  }
  pl->h_cur = 0;
  pl->h_counts = pl->h_buf[0];
  pl->topo = TunaTopo{P, l, g, elem_size};
  pl->radix_l = radix;
  pl->radix_g = (g > 1 && block_count == 0) ? radix_global : 2;
  pl->block_count = block_count;
  pl->flags = flags;
  pl->classic = (flags & TUNA_FLAG_CLASSIC_ROTATE) != 0;
  add_level(pl, 0, l, radix, g);
  if (g > 1 && block_count > 0)
    add_staggered(pl, block_count);
  else if (g > 1)
    add_level(pl, 1, g, pl->radix_g, l);

  const int64_t PP = (int64_t)P * P;
  const int nph = (int)pl->phases.size();
  cudaStream_t st = (cudaStream_t)stream;
  auto fail = [&](int code) {
    tuna_plan_destroy(pl);
    return code;
  };
#define TUNA_TRY(call)                                  \
  do {                                                  \
    cudaError_t e_ = (call);                            \
    if (e_ != cudaSuccess) {                            \
      int code_ = e_ == cudaErrorMemoryAllocation ? TUNA_ERR_NOMEM : TUNA_ERR_CUDA; \
      (void)cudaGetLastError();                         \
      return fail(code_);                               \
    }                                                   \
  } while (0)
  TUNA_TRY(dev_alloc(&pl->d_counts_buf[0], PP));
  TUNA_TRY(dev_alloc(&pl->d_counts_buf[1], PP));
  pl->d_counts = pl->d_counts_buf[0];
  TUNA_TRY(dev_alloc(&pl->d_sdispls, PP));
  TUNA_TRY(dev_alloc(&pl->d_rdispls, PP));
  TUNA_TRY(dev_alloc(&pl->d_sendbase, P));
  TUNA_TRY(dev_alloc(&pl->d_recvbase, P));
  for (int i = 0; i < 2; i++) {
    TUNA_TRY(dev_alloc(&pl->d_sz[i], PP));
    TUNA_TRY(dev_alloc(&pl->d_loc[i], PP));
  }
  TUNA_TRY(dev_alloc(&pl->d_seg_total, 2 * P));
  TUNA_TRY(dev_alloc(&pl->d_seg_raw, 2 * P));
  TUNA_TRY(dev_alloc(&pl->d_seg_base, 2 * P));
  TUNA_TRY(dev_alloc(&pl->d_tmp, PP));
  {
    const int64_t n_scal = 2 * (2 * nph + 3), n_wbase = nph + 1, n_ext = 6;  // ext [4], [5]: the row exchange's buffers
    const int64_t n_rb = std::max<int64_t>(pl->stats_n, 1), n_viol = 1 + 2 * nph + 3;
    pl->readback_words = n_scal + n_wbase + n_ext + n_rb + n_viol;
    TUNA_TRY(dev_alloc(&pl->d_readback, pl->readback_words));
    TUNA_TRY(cudaMemset(pl->d_readback, 0, (size_t)pl->readback_words * 8));
    if (cudaHostAlloc((void **)&pl->h_readback, (size_t)pl->readback_words * 8, cudaHostAllocDefault) != cudaSuccess) {
      (void)cudaGetLastError();
      pl->h_readback = nullptr;  // (the copies then go to pageable memory, one by one)
    }
    pl->d_scal = pl->d_readback;
    pl->d_wbase = pl->d_scal + n_scal;
    pl->d_extents = pl->d_wbase + n_wbase;
    pl->d_round_bytes = reinterpret_cast<unsigned long long *>(pl->d_extents + n_ext);
    pl->d_violations = pl->d_round_bytes + n_rb;
  }
  TUNA_TRY(dev_alloc(&pl->d_error, 1));
  TUNA_TRY(cudaMemset(pl->d_error, 0, sizeof(int)));
  pl->keep.resize(nph);
  pl->deliver.resize(nph);
  auto nomem = [&](int code) {
    return fail(pl->cuda_err == (int)cudaErrorMemoryAllocation ? TUNA_ERR_NOMEM : code);
  };
  for (int f = 0; f < nph; f++) {
    const TunaPhase &ph = pl->phases[f];
    rc = alloc_list(pl, pl->keep[f], TUNA_LIST_KEEP, (int64_t)P * (ph.per_rank - ph.finals));
    if (rc) return nomem(rc);
    rc = alloc_list(pl, pl->deliver[f], TUNA_LIST_DELIVER, (int64_t)P * ph.finals);
    if (rc) return nomem(rc);
  }
  rc = alloc_list(pl, pl->rot, TUNA_LIST_DELIVER, pl->classic ? PP : P);
  if (rc) return nomem(rc);
  pl->dir_shared = !pl->classic && g == 1 && block_count == 0 && nph == 1 &&
                   pl->phases[0].finals == pl->phases[0].per_rank;
  pl->no_direct = (flags & TUNA_FLAG_NO_DIRECT) != 0 && !pl->dir_shared;
  if (!pl->dir_shared && !pl->no_direct) {
    rc = alloc_list(pl, pl->dir, TUNA_LIST_DELIVER, PP);
    if (rc) return nomem(rc);
  }
  {  // the self-check's view of the lists: their arrays never move
    std::vector<TunaCheckItem> items;
    auto add = [&](const TunaList &l, int keep_phase, int id) {
      if (l.n <= 0) return;
      items.push_back(TunaCheckItem{l.len, l.pos, l.src, l.kind == TUNA_LIST_DELIVER ? l.dst : nullptr, l.n,
                                    keep_phase, id});
      pl->check_max_n = std::max(pl->check_max_n, l.n);
    };
    for (int f = 0; f < nph; f++) {
      add(pl->keep[f], f, f);
      add(pl->deliver[f], 0, nph + f);
    }
    add(pl->rot, 0, 2 * nph);
    if (!pl->dir_shared && !pl->no_direct) add(pl->dir, 0, 2 * nph + 1);
    pl->n_check_items = (int)items.size();
    if (!items.empty()) {
      TUNA_TRY(cudaMalloc(&pl->d_check_items, items.size() * sizeof(TunaCheckItem)));
      TUNA_TRY(cudaMemcpy(pl->d_check_items, items.data(), items.size() * sizeof(TunaCheckItem), cudaMemcpyHostToDevice));
    }
  }
#undef TUNA_TRY
  rc = build_tables(pl, &hl, sdispls, rdispls, st);
  if (rc) return fail(rc);
  *out = pl;
  return TUNA_OK;
}

int tuna_plan_create(tuna_plan_t **out, int P, int radix, int radix_global, int l, int g,
                     int elem_size, unsigned flags, const int64_t *sendcounts,
                     const int64_t *sdispls, const int64_t *rdispls, const int64_t *sendbase,
                     const int64_t *recvbase, void *stream) {
  return plan_create(out, P, radix, radix_global, 0, l, g, elem_size, flags, sendcounts, sdispls,
                     rdispls, sendbase, recvbase, stream);
}

int tuna_plan_create_staggered(tuna_plan_t **out, int P, int radix, int block_count, int l, int g,
                               int elem_size, unsigned flags, const int64_t *sendcounts,
                               const int64_t *sdispls, const int64_t *rdispls,
                               const int64_t *sendbase, const int64_t *recvbase, void *stream) {
  if (block_count < 1) {
    if (out) *out = nullptr;
    return TUNA_ERR_INVALID_ARG;
  }
  return plan_create(out, P, radix, 2, block_count, l, g, elem_size, flags, sendcounts, sdispls,
                     rdispls, sendbase, recvbase, stream);
}

int tuna_plan_update_counts(tuna_plan_t *pl, const int64_t *sendcounts, const int64_t *sdispls,
                            const int64_t *rdispls, const int64_t *sendbase,
                            const int64_t *recvbase, void *stream) {
  if (!pl || !sendcounts) return TUNA_ERR_INVALID_ARG;
  HostLayout hl;
  const int spare = pl->h_cur ^ 1;
  CountUpload up;  // the spare device buffer takes the new counts while the pass is running
  up.d_dst = pl->d_counts == pl->d_counts_buf[0] ? pl->d_counts_buf[1] : pl->d_counts_buf[0];
  up.st = (cudaStream_t)stream;
  const int rc = host_layout(pl->topo.P, sendcounts, sdispls, rdispls, sendbase, recvbase, &hl,
                             pl->h_buf[spare], &up);
  if (rc) {  // the plan still holds its previous counts, on the host and on the device
    if (rc == TUNA_ERR_CUDA) pl->cuda_err = (int)up.err;
    return rc;
  }
  pl->h_cur = spare;
  pl->h_counts = pl->h_buf[spare];
  if (up.done) {
    pl->d_counts = up.d_dst;
    pl->counts_uploaded = true;
  }
  return build_tables(pl, &hl, sdispls, rdispls, (cudaStream_t)stream);
}

int tuna_plan_update_counts_device(tuna_plan_t *pl, const int64_t *d_sendcounts, void *stream) {
  if (!pl || !d_sendcounts) return TUNA_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const int64_t PP = (int64_t)pl->topo.P * pl->topo.P;
  // the plan keeps its own copy (the caller may reuse its array at once), in the
  // buffer its tables were last built from: the kernels that read it stay the same
  {
    const int wrc = wait_in_flight(pl);
    if (wrc) return wrc;
  }
  pl->tables_valid = false;
  TUNA_CUDA(pl, cudaMemcpyAsync(pl->d_counts, d_sendcounts, (size_t)PP * 8, cudaMemcpyDeviceToDevice, st));
  return build_tables(pl, nullptr, nullptr, nullptr, st);
}

int tuna_plan_workspace_bytes(const tuna_plan_t *pl, size_t *bytes) {
  if (!pl || !bytes) return TUNA_ERR_INVALID_ARG;
  *bytes = (size_t)pl->workspace_need;
  return TUNA_OK;
}

int tuna_plan_host_staging_bytes(const tuna_plan_t *pl, size_t *bytes) {
  if (!pl || !bytes) return TUNA_ERR_INVALID_ARG;
  *bytes = (size_t)(align256(pl->send_extent) + align256(pl->recv_extent) + 256);
  return TUNA_OK;
}

int tuna_plan_set_workspace(tuna_plan_t *pl, void *dev_ptr, size_t bytes) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  if (dev_ptr && ((uintptr_t)dev_ptr & 255)) return TUNA_ERR_WORKSPACE;
  pl->workspace = (char *)dev_ptr;
  pl->workspace_bytes = dev_ptr ? bytes : 0;
  return TUNA_OK;
}

int tuna_plan_extents(const tuna_plan_t *pl, size_t *send_bytes, size_t *recv_bytes,
                      size_t *payload_bytes) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  if (send_bytes) *send_bytes = (size_t)pl->send_extent;
  if (recv_bytes) *recv_bytes = (size_t)pl->recv_extent;
  if (payload_bytes) *payload_bytes = (size_t)pl->payload;
  return TUNA_OK;
}

int tuna_alltoallv(tuna_plan_t *pl, const void *sendbuf, const int64_t *sendcounts,
                   const int64_t *sdispls, void *recvbuf, const int64_t *recvcounts,
                   const int64_t *rdispls, void *stream) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  if ((!sendbuf && pl->send_extent > 0) || (!recvbuf && pl->recv_extent > 0)) return TUNA_ERR_INVALID_ARG;
  int rc = check_call_args(pl, sendcounts, sdispls, recvcounts, rdispls);
  if (rc) return rc;
  if (ranges_overlap(sendbuf, (size_t)pl->send_extent, recvbuf, (size_t)pl->recv_extent))
    return TUNA_ERR_OVERLAP;
  return run_tuna(pl, sendbuf, recvbuf, (cudaStream_t)stream);
}

int tuna_direct_alltoallv(tuna_plan_t *pl, const void *sendbuf, const int64_t *sendcounts,
                          const int64_t *sdispls, void *recvbuf, const int64_t *recvcounts,
                          const int64_t *rdispls, void *stream) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  if ((!sendbuf && pl->send_extent > 0) || (!recvbuf && pl->recv_extent > 0)) return TUNA_ERR_INVALID_ARG;
  int rc = check_call_args(pl, sendcounts, sdispls, recvcounts, rdispls);
  if (rc) return rc;
  if (ranges_overlap(sendbuf, (size_t)pl->send_extent, recvbuf, (size_t)pl->recv_extent))
    return TUNA_ERR_OVERLAP;
  return run_direct(pl, sendbuf, recvbuf, (cudaStream_t)stream);
}

// Device-side alias of a pinned, mapped host buffer, or nullptr if the kernels
// cannot address it (pageable memory, or a null / empty buffer).
static void *mapped_alias(const void *host) {
  if (!host) return nullptr;
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
    (void)cudaGetLastError();
    return nullptr;
  }
  if (at.type != cudaMemoryTypeHost || !at.devicePointer) return nullptr;
  return at.devicePointer;
}

int tuna_alltoallv_host(tuna_plan_t *pl, const void *host_send, void *host_recv, int schedule,
                        void *stream) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  if ((!host_send && pl->send_extent > 0) || (!host_recv && pl->recv_extent > 0)) return TUNA_ERR_INVALID_ARG;
  const bool force_staging = (schedule & TUNA_HOST_STAGED) != 0;
  schedule &= ~TUNA_HOST_STAGED;
  if (schedule != TUNA_SCHEDULE_TUNA && schedule != TUNA_SCHEDULE_DIRECT) return TUNA_ERR_INVALID_ARG;
  if (!pl->tables_valid) return TUNA_ERR_INTERNAL;
  if (ranges_overlap(host_send, (size_t)pl->send_extent, host_recv, (size_t)pl->recv_extent))
    return TUNA_ERR_OVERLAP;
  cudaStream_t st = (cudaStream_t)stream;
  // Pinned, mapped host buffers: the kernels read the send buffer and write the
  // receive buffer in place, so the two directions of the host link run at the
  // same time and no block is copied twice.
  const int64_t w = align256(pl->workspace_need);
  const int64_t need = w + align256(pl->send_extent) + align256(pl->recv_extent) + 256;
  const bool can_stage = pl->workspace && pl->workspace_bytes >= (size_t)need;
  // Tiny blocks make poor use of the host link when the kernels touch them one by
  // one (measured: 0.6x of the staged path at 180-byte blocks, 1.3x at 2 MiB
  // blocks), so they are staged whenever the workspace has room for it.
  const int64_t blocks = (int64_t)pl->topo.P * pl->topo.P;
  const bool prefer_staging = pl->payload / blocks < kHostStagingBlockBytes && can_stage;
  if (!force_staging && !prefer_staging) {
    void *zs = pl->send_extent > 0 ? mapped_alias(host_send) : (void *)host_send;
    void *zr = pl->recv_extent > 0 ? mapped_alias(host_recv) : host_recv;
    if ((zs || pl->send_extent == 0) && (zr || pl->recv_extent == 0))
      return schedule == TUNA_SCHEDULE_TUNA ? run_tuna(pl, zs, zr, st) : run_direct(pl, zs, zr, st);
  }
  if (!can_stage) return TUNA_ERR_WORKSPACE;
  char *d_send = pl->workspace + w;
  char *d_recv = d_send + align256(pl->send_extent);
  if (pl->send_extent > 0)
    TUNA_CUDA(pl, cudaMemcpyAsync(d_send, host_send, (size_t)pl->send_extent, cudaMemcpyHostToDevice, st));
  int rc = schedule == TUNA_SCHEDULE_TUNA ? run_tuna(pl, d_send, d_recv, st)
                                          : run_direct(pl, d_send, d_recv, st);
  if (rc) return rc;
  if (pl->recv_extent > 0)
    TUNA_CUDA(pl, cudaMemcpyAsync(host_recv, d_recv, (size_t)pl->recv_extent, cudaMemcpyDeviceToHost, st));
  return TUNA_OK;
}

int tuna_plan_set_row_maps(tuna_plan_t *pl, const int64_t *gather_rows, const int64_t *scatter_rows,
                           int64_t in_rows, int64_t out_rows, void *stream) {
  if (!pl || in_rows < 0 || out_rows < 0) return TUNA_ERR_INVALID_ARG;
  if (!pl->tables_valid) return TUNA_ERR_INTERNAL;
  cudaStream_t st = (cudaStream_t)stream;
  const TunaTopo &t = pl->topo;
  const int P = t.P;
  const int64_t PP = (int64_t)P * P;
  const int64_t n = pl->payload / t.elem;  // rows exchanged
  {
    const int wrc = wait_in_flight(pl);  // a row exchange still running reads the list rewritten below
    if (wrc) return wrc;
  }
  pl->rows_valid = false;
  if (in_rows > (INT64_MAX >> 8) / t.elem || out_rows > (INT64_MAX >> 8) / t.elem) return TUNA_ERR_RANGE;
  if (!pl->d_row_start) TUNA_CUDA(pl, dev_alloc(&pl->d_row_start, PP));
  if (!pl->rowsl.len || n > pl->rows_cap) {
    free_list(pl->rowsl);
    pl->rows_cap = 0;
    const int rc = alloc_list(pl, pl->rowsl, TUNA_LIST_DELIVER, n);
    if (rc) return pl->cuda_err == (int)cudaErrorMemoryAllocation ? TUNA_ERR_NOMEM : rc;
    pl->rows_cap = n;
  }
  TunaList &l = pl->rowsl;
  l.n = n;
  const int th = 256;
  const unsigned gPP = (unsigned)((PP + th - 1) / th);
  const unsigned gseg = (unsigned)(((int64_t)P * 32 + th - 1) / th);
  const int nph = (int)pl->phases.size();
  Timed plan_timer(pl, TUNA_TIMER_PLAN, 0, st);
  // rows before every block in receive-side order: scan of the transposed counts
  tuna_transpose_kernel<<<dim3((P + 31) / 32, (P + 31) / 32), dim3(32, 8), 0, st>>>(pl->d_counts, pl->d_tmp, P, nullptr);
  TUNA_LAUNCHED(pl);
  tuna_segscan_kernel<0><<<gseg, th, 0, st>>>(pl->d_tmp, pl->d_row_start, pl->d_seg_total, nullptr, P, P);
  TUNA_LAUNCHED(pl);
  tuna_segbase_kernel<<<1, 1024, 0, st>>>(pl->d_seg_total, nullptr, pl->d_seg_base, P,
                                          pl->d_scal + 2 * (2 * nph + 2), nullptr, 0, nullptr, 0);
  TUNA_LAUNCHED(pl);
  tuna_add_base_kernel<<<gPP, th, 0, st>>>(pl->d_row_start, pl->d_seg_base, P, PP);
  TUNA_LAUNCHED(pl);
  const int64_t warps = PP;
  tuna_rows_list_kernel<<<(unsigned)((warps * 32 + th - 1) / th), th, 0, st>>>(
      P, t.elem, pl->d_counts, pl->d_sdispls, pl->d_rdispls, pl->d_sendbase, pl->d_recvbase,
      pl->d_row_start, gather_rows, scatter_rows, in_rows, out_rows, n, l.len, l.pos, l.src, l.dst);
  TUNA_LAUNCHED(pl);
  pl->rows_in_bytes = in_rows * t.elem;
  pl->rows_out_bytes = out_rows * t.elem;
  l.bytes = n * t.elem;
  l.total = n * (((int64_t)t.elem + 15) / 16 * 16 + 16);
  // every row must lie inside the two buffers
  const int64_t row_ext[2] = {pl->rows_in_bytes, pl->rows_out_bytes};
  TUNA_CUDA(pl, cudaMemcpyAsync(pl->d_extents + 4, row_ext, sizeof(row_ext), cudaMemcpyHostToDevice, st));
  TUNA_CUDA(pl, cudaMemsetAsync(pl->d_violations, 0, 2 * sizeof(unsigned long long), st));
  if (n > 0) {
    tuna_check_list_kernel<<<(unsigned)std::min<int64_t>((n + th - 1) / th, 148 * 8), th, 0, st>>>(
        l.len, l.pos, l.src, l.dst, n, pl->d_extents + 4, pl->d_wbase + nph, 0,
        pl->d_wbase, pl->d_violations, pl->d_violations + 1);
    TUNA_LAUNCHED(pl);
  }
  unsigned long long checked[2] = {0, 0};
  TUNA_CUDA(pl, cudaMemcpyAsync(checked, pl->d_violations, sizeof(checked), cudaMemcpyDeviceToHost, st));
  TUNA_CUDA(pl, cudaStreamSynchronize(st));
  if (checked[0] != 0) return TUNA_ERR_RANGE;
  l.unaligned_bytes = (int64_t)checked[1];
  int rc = build_chunks(pl, l, st);
  if (rc) return rc;
  rc = mark_tables_ready(pl, st);
  if (rc) return rc;
  pl->rows_valid = true;
  return TUNA_OK;
}

int tuna_rows_alltoallv(tuna_plan_t *pl, const void *rows_in, void *rows_out, void *stream) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  if (!pl->rows_valid) return TUNA_ERR_COUNT_MISMATCH;
  const TunaList &l = pl->rowsl;
  if (l.n > 0 && (!rows_in || !rows_out)) return TUNA_ERR_INVALID_ARG;
  if (ranges_overlap(rows_in, (size_t)pl->rows_in_bytes, rows_out, (size_t)pl->rows_out_bytes))
    return TUNA_ERR_OVERLAP;
  int launches = 0;
  cudaStream_t st = (cudaStream_t)stream;
  {
    const int arc = await_tables(pl, st);
    if (arc) return arc;
  }
  if (l.nchunks > 0) {
    Timed tm(pl, TUNA_TIMER_DIRECT, l.bytes, st);
    TunaMoveArgs a = move_args(pl, rows_in, rows_out, nullptr);
    a.extent[TUNA_BUF_SEND] = pl->rows_in_bytes;
    a.extent[TUNA_BUF_RECV] = pl->rows_out_bytes;
    a.del = list_args(l);
    TUNA_CUDA(pl, tuna_launch_move(TUNA_K_DIRECT, a, l.small_blocks, st));
    launches++;
  }
  pl->last_launches = launches;
  pl->launch_count += launches;
  return launches > 0 ? mark_in_flight(pl, st) : TUNA_OK;
}

int tuna_plan_num_rounds(const tuna_plan_t *pl, int *K) {
  if (!pl || !K) return TUNA_ERR_INVALID_ARG;
  *K = (int)pl->rounds.size();
  return TUNA_OK;
}

int tuna_plan_round_info(const tuna_plan_t *pl, int k, int *level, int *x, int *z, int64_t *units,
                         int64_t *bytes) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  if (k < 0 || k >= (int)pl->rounds.size()) return TUNA_ERR_RANGE;
  const auto &r = pl->rounds[k];
  if (level) *level = r.level;
  if (x) *x = r.x;
  if (z) *z = r.z;
  if (units) *units = r.units;
  if (bytes) *bytes = r.bytes;
  return TUNA_OK;
}

int tuna_plan_num_phases(const tuna_plan_t *pl, int *n) {
  if (!pl || !n) return TUNA_ERR_INVALID_ARG;
  *n = (int)pl->phases.size();
  return TUNA_OK;
}

static const TunaList *pick_list(const tuna_plan *pl, int phase, int part) {
  if (phase == -1) return &pl->rot;
  if (phase == -2) return &pl->dir;
  if (phase < 0 || phase >= (int)pl->phases.size()) return nullptr;
  if (part == TUNA_PART_KEEP) return &pl->keep[phase];
  if (part == TUNA_PART_DELIVER) return &pl->deliver[phase];
  return nullptr;
}

int tuna_plan_phase_info(const tuna_plan_t *pl, int phase, int part, int *level, int *x,
                         int64_t *entries, int64_t *bytes, int64_t *stream_bytes) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  const TunaList *l = pick_list(pl, phase, part);
  if (!l) return TUNA_ERR_RANGE;
  if (level) *level = phase >= 0 ? pl->phases[phase].level : -1;
  if (x) *x = phase >= 0 ? pl->phases[phase].x : -1;
  if (entries) *entries = l->n;
  if (bytes) *bytes = l->bytes;
  if (stream_bytes) *stream_bytes = l->total;
  return TUNA_OK;
}

int tuna_plan_phase_tables(const tuna_plan_t *pl, int phase, int part, int64_t cap, int64_t *len,
                           int64_t *pos, int64_t *src, int64_t *dst, int64_t *rows) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  const TunaList *l = pick_list(pl, phase, part);
  if (!l) return TUNA_ERR_RANGE;
  if (rows) *rows = l->n;
  const int64_t n = std::min(cap, l->n);
  if (n <= 0) return TUNA_OK;
  tuna_plan *m = const_cast<tuna_plan *>(pl);
  TUNA_CUDA(m, cudaDeviceSynchronize());
  if (len) TUNA_CUDA(m, cudaMemcpy(len, l->len, n * 8, cudaMemcpyDeviceToHost));
  if (pos) TUNA_CUDA(m, cudaMemcpy(pos, l->pos, n * 8, cudaMemcpyDeviceToHost));
  if (src) TUNA_CUDA(m, cudaMemcpy(src, l->src, n * 8, cudaMemcpyDeviceToHost));
  if (dst) {
    if (l->kind == TUNA_LIST_DELIVER) {
      TUNA_CUDA(m, cudaMemcpy(dst, l->dst, n * 8, cudaMemcpyDeviceToHost));
    } else {  // a KEEP list's stream is its destination: workspace offset of the phase + position
      std::vector<int64_t> p(n);
      TUNA_CUDA(m, cudaMemcpy(p.data(), l->pos, n * 8, cudaMemcpyDeviceToHost));
      for (int64_t i = 0; i < n; i++) dst[i] = TUNA_LOC(TUNA_BUF_WORK, pl->h_wbase[phase] + p[i]);
    }
  }
  return TUNA_OK;
}

int tuna_plan_last_launches(const tuna_plan_t *pl, int *launches) {
  if (!pl || !launches) return TUNA_ERR_INVALID_ARG;
  *launches = pl->last_launches;
  return TUNA_OK;
}

int tuna_plan_launch_count(const tuna_plan_t *pl, int64_t *launches) {
  if (!pl || !launches) return TUNA_ERR_INVALID_ARG;
  *launches = pl->launch_count;
  return TUNA_OK;
}

int tuna_plan_enable_timing(tuna_plan_t *pl, int on) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  pl->timing = on != 0;
  return TUNA_OK;
}

int tuna_plan_get_timing(tuna_plan_t *pl, int reset, double *ms, int64_t *launches, int64_t *bytes) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  for (auto &s : pl->stamps) {
    TUNA_CUDA(pl, cudaEventSynchronize(s.b));
    float t = 0.f;
    TUNA_CUDA(pl, cudaEventElapsedTime(&t, s.a, s.b));
    pl->t_ms[s.kind] += t;
    pl->t_launches[s.kind] += 1;
    pl->t_bytes[s.kind] += s.bytes;
    pl->event_pool.push_back(s.a);
    pl->event_pool.push_back(s.b);
  }
  pl->stamps.clear();
  for (int k = 0; k < TUNA_TIMER_KINDS; k++) {
    if (ms) ms[k] = pl->t_ms[k];
    if (launches) launches[k] = pl->t_launches[k];
    if (bytes) bytes[k] = pl->t_bytes[k];
    if (reset) {
      pl->t_ms[k] = 0;
      pl->t_launches[k] = 0;
      pl->t_bytes[k] = 0;
    }
  }
  return TUNA_OK;
}

int tuna_plan_cuda_error(const tuna_plan_t *pl) { return pl ? pl->cuda_err : 0; }

int tuna_plan_device_status(tuna_plan_t *pl, int *gave_up) {
  if (!pl || !gave_up) return TUNA_ERR_INVALID_ARG;
  TUNA_CUDA(pl, cudaDeviceSynchronize());
  TUNA_CUDA(pl, cudaMemcpy(gave_up, pl->d_error, sizeof(int), cudaMemcpyDeviceToHost));
  return TUNA_OK;
}

// ------------------------------------------------------------------ allocation-free direct exchange

}  // extern "C"

namespace {

// Scratch of tuna_direct_alltoallv_static: every table the direct exchange needs,
// for up to TUNA_STATIC_MAX_P ranks, in one file-scope device array.  The array
// exists once per GPU that loads the library and lives until the process ends.
constexpr int64_t kStaticPP = (int64_t)TUNA_STATIC_MAX_P * TUNA_STATIC_MAX_P;
constexpr int64_t kStaticWords = 8 * kStaticPP + 1      // counts, sdispls, rdispls, tmp, len, pos(+1), src, dst
                                 + 5 * TUNA_STATIC_MAX_P  // sendbase, recvbase, seg_total, seg_raw, seg_base
                                 + 2                      // stream totals
                                 + TUNA_STATIC_MAX_CHUNKS / 2 + 1;  // chunk table (32-bit entries)
static __device__ __align__(256) int64_t tuna_static_scratch[kStaticWords];

struct StaticTables {
  int64_t *counts, *sdispls, *rdispls, *tmp, *len, *pos, *src, *dst;
  int64_t *sendbase, *recvbase, *seg_total, *seg_raw, *seg_base, *scal;
  int32_t *chunk_first;
};

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
int64_t *g_static_ptr[kMaxDevices] = {};  // device address of the scratch, per device ordinal

// The array's name is only a host-side handle; kernels need its device address.
// Looked up once per device, with that device current.
cudaError_t static_tables(StaticTables *t) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  int64_t *base;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
      void *p = nullptr;
      e = cudaGetSymbolAddress(&p, tuna_static_scratch);
      if (e != cudaSuccess) return e;
      g_static_ptr[dev] = (int64_t *)p;
    }
    base = g_static_ptr[dev];
  }
  int64_t *w = base;
  auto take = [&](int64_t n) {
    int64_t *r = w;
    w += n;
    return r;
  };
  t->counts = take(kStaticPP);
  t->sdispls = take(kStaticPP);
  t->rdispls = take(kStaticPP);
  t->tmp = take(kStaticPP);
  t->len = take(kStaticPP);
  t->pos = take(kStaticPP + 1);
  t->src = take(kStaticPP);
  t->dst = take(kStaticPP);
  t->sendbase = take(TUNA_STATIC_MAX_P);
  t->recvbase = take(TUNA_STATIC_MAX_P);
  t->seg_total = take(TUNA_STATIC_MAX_P);
  t->seg_raw = take(TUNA_STATIC_MAX_P);
  t->seg_base = take(TUNA_STATIC_MAX_P);
  t->scal = take(2);
  t->chunk_first = (int32_t *)take(TUNA_STATIC_MAX_CHUNKS / 2 + 1);
  return cudaSuccess;
}

// Descriptors of the direct exchange in receive-side order (d, s).
__global__ void tuna_static_direct_list_kernel(int P, int elem, const int64_t *__restrict__ counts,
                                               const int64_t *__restrict__ sdispls,
                                               const int64_t *__restrict__ rdispls,
                                               const int64_t *__restrict__ sendbase,
                                               const int64_t *__restrict__ recvbase, int64_t *len,
                                               int64_t *src, int64_t *dst) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)P * P) return;
  const int d = (int)(idx / P), s = (int)(idx % P);
  len[idx] = counts[(int64_t)s * P + d] * elem;
  src[idx] = TUNA_LOC(TUNA_BUF_SEND, (sendbase[s] + sdispls[(int64_t)s * P + d]) * elem);
  dst[idx] = TUNA_LOC(TUNA_BUF_RECV, (recvbase[d] + rdispls[(int64_t)d * P + s]) * elem);
}

}  // namespace

extern "C" {

int tuna_direct_alltoallv_static(int P, int elem_size, const int64_t *sendcounts,
                                 const int64_t *sdispls, const int64_t *rdispls,
                                 const int64_t *sendbase, const int64_t *recvbase,
                                 const void *sendbuf, void *recvbuf, void *stream) {
  if (P < 1 || elem_size < 1 || !sendcounts) return TUNA_ERR_INVALID_ARG;
  if (P > TUNA_STATIC_MAX_P) return TUNA_ERR_RANGE;
  int rc = validate_layout(P, sendcounts, sdispls, rdispls, sendbase, recvbase);
  if (rc) return rc;
  const int64_t PP = (int64_t)P * P;
  // host side: region bases, extents, and the length of the work stream
  int64_t sb[TUNA_STATIC_MAX_P], rb[TUNA_STATIC_MAX_P], sreg[TUNA_STATIC_MAX_P], rreg[TUNA_STATIC_MAX_P];
  for (int p = 0; p < P; p++) sreg[p] = rreg[p] = 0;
  int64_t stream_bytes = 0, payload = 0;
  for (int s = 0; s < P; s++)
    for (int d = 0; d < P; d++) {
      const int64_t c = sendcounts[(int64_t)s * P + d];
      const int64_t bytes = c * elem_size;
      payload += bytes;
      if (bytes > 0) stream_bytes += ((bytes + 15) & ~(int64_t)15) + 16;
      if (sdispls) sreg[s] = std::max(sreg[s], sdispls[(int64_t)s * P + d] + c); else sreg[s] += c;
      if (rdispls) rreg[d] = std::max(rreg[d], rdispls[(int64_t)d * P + s] + c); else rreg[d] += c;
    }
  int64_t se = 0, re = 0, acc_s = 0, acc_r = 0;
  for (int p = 0; p < P; p++) {
    sb[p] = sendbase ? sendbase[p] : acc_s;
    rb[p] = recvbase ? recvbase[p] : acc_r;
    acc_s += sreg[p];
    acc_r += rreg[p];
    se = std::max(se, sb[p] + sreg[p]);
    re = std::max(re, rb[p] + rreg[p]);
  }
  se *= elem_size;
  re *= elem_size;
  if ((!sendbuf && se > 0) || (!recvbuf && re > 0)) return TUNA_ERR_INVALID_ARG;
  if (ranges_overlap(sendbuf, (size_t)se, recvbuf, (size_t)re)) return TUNA_ERR_OVERLAP;
  if (payload == 0) return TUNA_OK;
  int64_t chunk = 8192;
  while (chunk < TUNA_MAX_CHUNK_BYTES &&
         ((chunk < 65536 && stream_bytes / chunk > 148 * 32) ||
          (stream_bytes + chunk - 1) / chunk > TUNA_STATIC_MAX_CHUNKS))
    chunk <<= 1;
  const int64_t nchunks = (stream_bytes + chunk - 1) / chunk;
  if (nchunks > TUNA_STATIC_MAX_CHUNKS) return TUNA_ERR_RANGE;  // more than 4 GiB of work stream

  StaticTables t;
  if (static_tables(&t) != cudaSuccess) return TUNA_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
#define TUNA_STATIC_CUDA(call)              \
  do {                                      \
    if ((call) != cudaSuccess) return TUNA_ERR_CUDA; \
  } while (0)
  const int th = 256;
  const unsigned gPP = (unsigned)((PP + th - 1) / th);
  const unsigned gseg = (unsigned)(((int64_t)P * 32 + th - 1) / th);
  TUNA_STATIC_CUDA(cudaMemcpyAsync(t.counts, sendcounts, PP * 8, cudaMemcpyHostToDevice, st));
  TUNA_STATIC_CUDA(cudaMemcpyAsync(t.sendbase, sb, P * 8, cudaMemcpyHostToDevice, st));
  TUNA_STATIC_CUDA(cudaMemcpyAsync(t.recvbase, rb, P * 8, cudaMemcpyHostToDevice, st));
  if (sdispls) {
    TUNA_STATIC_CUDA(cudaMemcpyAsync(t.sdispls, sdispls, PP * 8, cudaMemcpyHostToDevice, st));
  } else {
    tuna_segscan_kernel<0><<<gseg, th, 0, st>>>(t.counts, t.sdispls, t.seg_total, nullptr, P, P);
    TUNA_STATIC_CUDA(cudaGetLastError());
  }
  if (rdispls) {
    TUNA_STATIC_CUDA(cudaMemcpyAsync(t.rdispls, rdispls, PP * 8, cudaMemcpyHostToDevice, st));
  } else {
    tuna_transpose_kernel<<<dim3((P + 31) / 32, (P + 31) / 32), dim3(32, 8), 0, st>>>(t.counts, t.tmp, P, nullptr);
    TUNA_STATIC_CUDA(cudaGetLastError());
    tuna_segscan_kernel<0><<<gseg, th, 0, st>>>(t.tmp, t.rdispls, t.seg_total, nullptr, P, P);
    TUNA_STATIC_CUDA(cudaGetLastError());
  }
  tuna_static_direct_list_kernel<<<gPP, th, 0, st>>>(P, elem_size, t.counts, t.sdispls, t.rdispls,
                                                     t.sendbase, t.recvbase, t.len, t.src, t.dst);
  TUNA_STATIC_CUDA(cudaGetLastError());
  tuna_segscan_kernel<2><<<gseg, th, 0, st>>>(t.len, t.pos, t.seg_total, t.seg_raw, P, P);
  TUNA_STATIC_CUDA(cudaGetLastError());
  tuna_segbase_kernel<<<1, 1024, 0, st>>>(t.seg_total, t.seg_raw, t.seg_base, P, t.scal, nullptr, 0,
                                          t.pos + PP, 0);
  TUNA_STATIC_CUDA(cudaGetLastError());
  tuna_add_base_kernel<<<gPP, th, 0, st>>>(t.pos, t.seg_base, P, PP);
  TUNA_STATIC_CUDA(cudaGetLastError());
  tuna_chunk_index_kernel<<<(unsigned)((nchunks + 128) / 128), 128, 0, st>>>(t.pos, PP, chunk, nchunks,
                                                                             stream_bytes, t.chunk_first);
  TUNA_STATIC_CUDA(cudaGetLastError());
  TunaMoveArgs a{};
  a.del.len = t.len;
  a.del.pos = t.pos;
  a.del.src = t.src;
  a.del.dst = t.dst;
  a.del.chunk_first = t.chunk_first;
  a.del.n = PP;
  a.del.total = stream_bytes;
  a.del.chunk = chunk;
  a.del.nchunks = nchunks;
  a.base[TUNA_BUF_SEND] = (char *)const_cast<void *>(sendbuf);
  a.base[TUNA_BUF_RECV] = (char *)recvbuf;
  a.base[TUNA_BUF_WORK] = nullptr;
  a.extent[TUNA_BUF_SEND] = se;
  a.extent[TUNA_BUF_RECV] = re;
  a.extent[TUNA_BUF_WORK] = 0;
  TUNA_STATIC_CUDA(tuna_launch_move(TUNA_K_DIRECT, a, payload / PP < kStaticSmallBlockBytes, st));
#undef TUNA_STATIC_CUDA
  return TUNA_OK;
}

}  // extern "C"

