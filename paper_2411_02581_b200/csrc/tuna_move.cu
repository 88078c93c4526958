// Fused pack-move-unpack kernels.
//
// One launch executes every copy descriptor of one list.  A digit phase of the
// radix-r schedule (all rounds z of one digit position x: the blocks whose x-th
// offset digit equals z leave the rank that holds them for the rank at distance
// +z*r^x; Sec. III-A/B of the paper) has two lists: the blocks that travel on
// afterwards (KEEP: they land, in slot order, in that phase's region of the
// workspace) and the blocks that have arrived (DELIVER: they land in the
// receive buffer at their MPI_Alltoallv displacement).  The final rotation and
// the single-pass direct exchange (Sec. II-d) are DELIVER lists too.  "Pack" is
// the gather from the source rank's buffer, "move" the rank shift, "unpack" the
// placement at the destination; with all ranks in one memory the three are one
// copy, so each payload byte is read once and written once per hop.
//
// Work is partitioned by bytes, not by blocks: a list's stream (its blocks in
// receive-side order, padded to 16 bytes) is cut into equal chunks, one CTA per
// chunk, and a precomputed table gives the first descriptor of every chunk.  A
// block larger than a chunk is spread over several CTAs; a chunk of tiny blocks
// is shared out over the threads of one CTA, which walk the chunk as one run of
// 16-byte vectors: a small table in shared memory says which block owns which
// vector, so that consecutive threads copy consecutive vectors whatever the
// block boundaries are, several loads in flight per thread before the first store.
//
// A launch carries up to three independent lists (the block index picks list and
// chunk): a digit phase is ONE tuna_round_kernel launch over its KEEP list, its
// DELIVER list and, in the first phase, the self blocks; tuna_rotate_kernel runs a
// rotation list alone (classic mode), tuna_direct_kernel the direct list.
//
//   KEEP lists.          The stream IS the destination, so stores
//                        are contiguous aligned vectors (a block's padding is
//                        written too: it is the library's own memory); sources are
//                        aligned workspace blocks or arbitrarily aligned
//                        send-buffer blocks (read as aligned words merged by
//                        funnel shifts).
//   DELIVER lists.       The stream spaces the blocks so that
//                        block e can be thought of as sitting at its destination's
//                        alignment: vector v of the stream then corresponds to
//                        one 16-byte aligned vector of the destination.  Vectors
//                        that lie wholly inside a block are stored as such; the
//                        partial first and last vector of each block are written
//                        afterwards by the block's own thread, in the widest
//                        aligned pieces that fit.  No byte outside a block's
//                        destination range is written.
// No byte outside a source buffer's extent is read: blocks within 31 bytes of
// either end of their buffer are read byte by byte instead of by aligned windows.
#include <stdlib.h>

#include "tuna_internal.h"

namespace {

constexpr int kThreads = TUNA_MOVE_THREADS;
constexpr int kBatch = kThreads;        // descriptors handled per batch (one per thread)
constexpr int kClampVec = 1 << 26;      // |vector index| beyond which only "far away" matters

__device__ __forceinline__ uint4 ld16(const char *p) { return *reinterpret_cast<const uint4 *>(p); }
__device__ __forceinline__ void st16(char *p, uint4 v) { *reinterpret_cast<uint4 *>(p) = v; }

// (a select, not an index: indexing a kernel parameter array spills it to local memory)
__device__ __forceinline__ char *base_of(const TunaMoveArgs &a, int buf) {
  if (buf >= TUNA_BUF_PEER0) return a.peer[buf - TUNA_BUF_PEER0];  // another GPU's receive buffer (sharded plans)
  return buf == TUNA_BUF_SEND ? a.base[0] : (buf == TUNA_BUF_RECV ? a.base[1] : a.base[2]);
}
__device__ __forceinline__ int64_t extent_of(const TunaMoveArgs &a, int buf) {
  return buf == TUNA_BUF_SEND ? a.extent[0] : (buf == TUNA_BUF_RECV ? a.extent[1] : a.extent[2]);
}

// Largest t < cnt with start[t] <= v (start is non-decreasing, start[0] <= v).
// Branch-free: eight select steps.
__device__ __forceinline__ int find_entry(const int *start, int cnt, int v) {
  int lo = 0;
#pragma unroll
  for (int step = kBatch / 2; step > 0; step >>= 1) {
    const int i = lo + step;
    const bool in = i < cnt;
    lo = (in && start[in ? i : 0] <= v) ? i : lo;
  }
  return lo;
}

// Owner table: who[v] = the descriptor (index in the batch) owning chunk vector v,
// for v in [vlo, vhi).  Every descriptor with vectors has already written its index
// at its first vector into the zeroed table; what is left is a running maximum
// (indices grow with position).  Each thread takes a run of vectors, starts from
// the owner of the run's first vector (one binary search) and sweeps four table
// bytes at a time with packed byte maxima.
__device__ __forceinline__ void fill_owner(unsigned char *who, const int *start, int cnt, int vlo,
                                           int vhi) {
  const int a0 = vlo & ~3;
  const int span = (((vhi - a0) + kThreads - 1) / kThreads + 3) & ~3;
  const int v0 = a0 + (int)threadIdx.x * span;
  if (v0 >= vhi) return;
  const int vend = (v0 + span < vhi) ? v0 + span : vhi;
  unsigned carry = (unsigned)find_entry(start, cnt, v0 > vlo ? v0 : vlo);
  for (int v = v0; v < vend; v += 4) {
    unsigned w = *reinterpret_cast<unsigned *>(who + v);
    w = __vmaxu4(w, carry);    // the owner so far enters at byte 0
    w = __vmaxu4(w, w << 8);   // prefix maximum over the four bytes
    w = __vmaxu4(w, w << 16);
    *reinterpret_cast<unsigned *>(who + v) = w;
    carry = w >> 24;
  }
}

// The 16 bytes at sa (any alignment) from the two 16-byte aligned vectors that hold them: word
// selection by the offset's bits 2 and 3, then funnel shifts by its low two bits.
// Two wide loads put far less load on the L1 data pipe than five aligned words
// would (a warp's 4-byte loads at a 16-byte stride use a quarter of every line
// they fetch).  Reads [sa - (sa & 15), +32).
__device__ __forceinline__ uint4 load16_pair(const char *sa) {
  const uintptr_t a = reinterpret_cast<uintptr_t>(sa);
  const uint4 *p = reinterpret_cast<const uint4 *>(a & ~(uintptr_t)15);
  const uint4 A = p[0], B = p[1];
  const bool j1 = (a & 4) != 0, j2 = (a & 8) != 0;
  const unsigned bits = (unsigned)(a & 3) * 8;
  const uint32_t u0 = j1 ? A.y : A.x, u1 = j1 ? A.z : A.y, u2 = j1 ? A.w : A.z, u3 = j1 ? B.x : A.w;
  const uint32_t u4 = j1 ? B.y : B.x, u5 = j1 ? B.z : B.y, u6 = j1 ? B.w : B.z;
  const uint32_t t0 = j2 ? u2 : u0, t1 = j2 ? u3 : u1, t2 = j2 ? u4 : u2, t3 = j2 ? u5 : u3, t4 = j2 ? u6 : u4;
  uint4 v;
  v.x = __funnelshift_r(t0, t1, bits);
  v.y = __funnelshift_r(t1, t2, bits);
  v.z = __funnelshift_r(t2, t3, bits);
  v.w = __funnelshift_r(t3, t4, bits);
  return v;
}

// Only the bytes [b0, b1) of the vector at sa, one by one (for blocks at the very
// ends of their source buffer, where an aligned window would leave it).
__device__ __noinline__ uint4 load16_bytes(const char *sa, int b0, int b1) {
  uint32_t w[4] = {0, 0, 0, 0};
  for (int i = b0; i < b1; i++) w[i >> 2] |= (uint32_t)(unsigned char)sa[i] << (8 * (i & 3));
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// Store bytes [b0, b1) of a vector parked in shared memory (sc, 16-byte aligned) to
// the 16-byte aligned global address gp, in the widest naturally aligned pieces
// that fit.  Every piece is a narrow shared load followed by a store of the same
// width, so no byte is shifted in registers.  Straight-line: pieces of 1, 2, 4, 8
// bytes while the position's alignment grows (each only if it still fits), then
// 8, 4, 2, 1 bytes for what is left.
__device__ __forceinline__ void store_pieces(char *gp, const unsigned char *sc, int b0, int b1) {
  int p = b0;
  if ((p & 1) && p + 1 <= b1) {
    *reinterpret_cast<unsigned char *>(gp + p) = *reinterpret_cast<const unsigned char *>(sc + p);
    p += 1;
  }
  if ((p & 2) && p + 2 <= b1) {
    *reinterpret_cast<unsigned short *>(gp + p) = *reinterpret_cast<const unsigned short *>(sc + p);
    p += 2;
  }
  if ((p & 4) && p + 4 <= b1) {
    *reinterpret_cast<uint32_t *>(gp + p) = *reinterpret_cast<const uint32_t *>(sc + p);
    p += 4;
  }
  if ((p & 8) && p + 8 <= b1) {
    *reinterpret_cast<unsigned long long *>(gp + p) = *reinterpret_cast<const unsigned long long *>(sc + p);
    p += 8;
  }
  // p is now aligned to every size that is still to come
  const int r = b1 - p;
  if (r & 8) {
    *reinterpret_cast<unsigned long long *>(gp + p) = *reinterpret_cast<const unsigned long long *>(sc + p);
    p += 8;
  }
  if (r & 4) {
    *reinterpret_cast<uint32_t *>(gp + p) = *reinterpret_cast<const uint32_t *>(sc + p);
    p += 4;
  }
  if (r & 2) {
    *reinterpret_cast<unsigned short *>(gp + p) = *reinterpret_cast<const unsigned short *>(sc + p);
    p += 2;
  }
  if (r & 1) *reinterpret_cast<unsigned char *>(gp + p) = *reinterpret_cast<const unsigned char *>(sc + p);
}

// ------------------------------------------------------------------ bulk copies (TMA)
//
// Optional route (TUNA_FLAG_BULK_COPY).  A chunk that lies inside one large aligned
// block needs no SM work at all: one thread hands it to the copy engine of the SM
// in pieces (cp.async.bulk, global ->
// shared, completion counted in bytes on an mbarrier) and, as each piece lands,
// sends it on (cp.async.bulk, shared -> global).  Addresses and sizes are
// multiples of 16 bytes by construction.  Every wait is bounded: if a barrier does
// not complete, the CTA raises the launch's error flag and leaves.  Measured on
// 2 MiB blocks this route reaches 6.58 TB/s against 6.65 TB/s for the plain vector
// loop (64 KiB of staging leave three CTAs per SM), so it is off by default.

constexpr int kBulkPiece = 16384;
constexpr int kBulkPieces = 4;                       // pieces in flight: one 64 KiB chunk
constexpr int kBulkBytes = kBulkPiece * kBulkPieces;
constexpr int kBulkMin = 16384;                      // shorter ranges are copied by the threads

__device__ __forceinline__ unsigned smem_u32(const void *p) {
  return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity) {
  for (int it = 0; it < (1 << 20); it++) {  // each try_wait sleeps for a while by itself
    unsigned ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void bulk_load(unsigned smem_dst, const void *gsrc, unsigned bytes, unsigned bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_dst),
               "l"(gsrc), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void bulk_store(void *gdst, unsigned smem_src, unsigned bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_src), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// waits until the committed stores have been written (not only read out of shared memory)
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ------------------------------------------------------------------ dependent launches
//
// The launches of one exchange form a chain on a stream.  From the second one on,
// each is launched with programmatic stream serialization: its CTAs may start
// while the previous launch is still draining, do their set-up (which reads only
// the plan's tables), and then block in hardware until the previous launch has
// completed and its writes are visible.  Every launch lets its successor start
// early right away.  The first launch after the plan's tables have been rewritten
// waits before it reads anything: what precedes it on the stream may be the plan
// kernels that write the very tables its set-up reads, and their stores are only
// guaranteed visible behind the wait (its CTAs are still scheduled early, which
// hides the launch latency).  Once one launch has run behind those kernels in
// full, the tables are settled and later exchanges start early again.

__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// ------------------------------------------------------------------ one skewed block
//
// A run of m whole vectors inside one block whose source is not 16-byte aligned
// (dst is).  Every output vector needs two neighbouring aligned source vectors;
// instead of loading both, a lane loads one and takes the other from the next lane
// by shuffle, so the loads are those of a plain copy.  A warp therefore turns 32
// loaded vectors into 31 stored ones; consecutive warp tiles overlap by one vector.
// The source's offset in its vector is the same for the whole run, so which words
// to merge is decided once (Q = offset / 4), outside the loop.
// Reads [src - (src & 15), src + 16 m + 16 - (src & 15)).
template <int kUnroll, int Q>
__device__ __forceinline__ void skewed_run_q(const uint4 *a0, unsigned bits, char *dst, int m) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kWarps = kThreads / 32;
  for (int g0 = warp; g0 * 31 < m; g0 += kUnroll * kWarps) {  // (warp-uniform: the shuffles need every lane)
    uint4 A[kUnroll];
#pragma unroll
    for (int k = 0; k < kUnroll; k++) {
      const int i = (g0 + k * kWarps) * 31 + lane;
      A[k] = i <= m ? a0[i] : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int k = 0; k < kUnroll; k++) {
      const int i = (g0 + k * kWarps) * 31 + lane;
      // words Q .. Q + 4 of the eight this lane and the next one hold
      uint32_t w[8];
      w[0] = A[k].x, w[1] = A[k].y, w[2] = A[k].z, w[3] = A[k].w;
#pragma unroll
      for (int j = 0; j <= Q; j++) {
        const uint32_t mine = j == 0 ? A[k].x : j == 1 ? A[k].y : j == 2 ? A[k].z : A[k].w;
        w[4 + j] = __shfl_down_sync(0xffffffffu, mine, 1);
      }
      uint4 x;
      x.x = __funnelshift_r(w[Q], w[Q + 1], bits);
      x.y = __funnelshift_r(w[Q + 1], w[Q + 2], bits);
      x.z = __funnelshift_r(w[Q + 2], w[Q + 3], bits);
      x.w = __funnelshift_r(w[Q + 3], w[Q + 4], bits);
      if (lane < 31 && i < m) st16(dst + ((int64_t)i << 4), x);
    }
  }
}

template <int kUnroll>
__device__ __forceinline__ void skewed_run(const char *src, char *dst, int m) {
  const unsigned sh = (unsigned)(reinterpret_cast<uintptr_t>(src) & 15);
  const uint4 *a0 = reinterpret_cast<const uint4 *>(src - sh);
  const unsigned bits = (sh & 3) * 8;
  switch (sh >> 2) {
    case 0: skewed_run_q<kUnroll, 0>(a0, bits, dst, m); break;
    case 1: skewed_run_q<kUnroll, 1>(a0, bits, dst, m); break;
    case 2: skewed_run_q<kUnroll, 2>(a0, bits, dst, m); break;
    default: skewed_run_q<kUnroll, 3>(a0, bits, dst, m); break;
  }
}

// ------------------------------------------------------------------ the mover

struct __align__(16) BlockPtrs {
  const char *sadj;
  char *dadj;
};

template <bool DELIVER, int kUnroll, bool kBulk>  // kUnroll: vectors a thread has in flight
__device__ __forceinline__ void move_body(const TunaListArgs &l, const TunaMoveArgs &a, int64_t c) {
  __shared__ int s_vs[kBatch];             // first vector of the block, relative to the chunk
  // per block of the batch: (DELIVER) the chunk-relative position of its first byte and
  // one past its last byte (clamped when far); the source address of chunk vector v
  // minus 16 v and (DELIVER) the destination address likewise (16-byte aligned).
  // Paired up so that a vector's look-up is one 8-byte and one 16-byte shared load.
  __shared__ int2 s_oe[DELIVER ? kBatch : 1];
  __shared__ BlockPtrs s_sd[kBatch];
  __shared__ unsigned char s_careful[kBatch];
  __shared__ __align__(16) unsigned char s_edge[DELIVER ? kBatch * 32 : 16];  // two parking slots per block: its partial first and last vector
  extern __shared__ __align__(16) unsigned char s_who[];  // owner of every vector of the chunk (chunk / 16 bytes)

  // bulk route (builds with kBulk only): barriers, their phase, the staging area behind the owner table
  __shared__ __align__(8) unsigned long long s_bar[kBulkPieces];
  __shared__ int s_abort;
  unsigned bulk_phase = 0;  // bit j: parity of barrier j's current phase
  bool bar_ready = false;
  bool waited = false;      // has this CTA waited for the previous launch of the stream yet?

  const int tid = threadIdx.x, lane = tid & 31;
  if (kBulk && tid == 0) s_abort = 0;
  const int64_t cA = c * l.chunk;
  const int64_t cB = (cA + l.chunk < l.total) ? cA + l.chunk : l.total;
  const int nv = (int)((cB - cA) >> 4);
  const int64_t e_lo = l.chunk_first[c];
  const int64_t e_hi = l.chunk_first[c + 1];  // the table has nchunks + 1 entries
  char *const keep_out = DELIVER ? nullptr : a.base[2] + a.keep_base + cA;

  for (int64_t b = e_lo; b <= e_hi; b += kBatch) {
    const int cnt = (int)((e_hi - b + 1 < kBatch) ? e_hi - b + 1 : kBatch);
    __syncthreads();  // the previous batch is done with the tables
    if (kBulk && s_abort) return;
    int my_org = 0, my_end = 0;
    bool my_edges = false;
    for (int i = tid * 16; i < nv + 4; i += kThreads * 16)  // the owner table starts out empty
      *reinterpret_cast<uint4 *>(s_who + i) = make_uint4(0, 0, 0, 0);
    int mark_at = -1;  // chunk vector at which this thread's block starts, if it has vectors in the chunk
    if (tid < cnt) {
      const int64_t e = b + tid;
      const int64_t p = l.pos[e];
      const int64_t s = l.src[e];
      const int sb = TUNA_LOC_BUF(s);
      const char *sbase = base_of(a, sb);
      const char *sp = sbase + TUNA_LOC_OFF(s);
      const int64_t rel = p - cA;
      int64_t vs = rel >> 4;
      if (vs < -kClampVec) vs = -kClampVec;
      s_vs[tid] = (int)vs;
      if (DELIVER) {
        const int64_t L = l.len[e];
        const int64_t d = l.dst[e];
        char *dp = base_of(a, TUNA_LOC_BUF(d)) + TUNA_LOC_OFF(d);
        const int ad = (int)(reinterpret_cast<uintptr_t>(dp) & 15);
        const int64_t org = rel + ad;  // exact chunk-relative position of byte 0
        int64_t end = org + L;
        if (end > ((int64_t)kClampVec << 4)) end = (int64_t)kClampVec << 4;
        my_org = (int)(vs << 4) + ad;
        my_end = (int)end;
        s_oe[tid] = make_int2(my_org, my_end);
        BlockPtrs ptrs;
        ptrs.sadj = sp - org;
        ptrs.dadj = dp - org;
        s_sd[tid] = ptrs;
        s_careful[tid] = (L > 0 && (sp - 31 < sbase || sp + L + 31 > sbase + extent_of(a, sb))) ? 1 : 0;
        my_edges = L > 0 && (ad != 0 || (L & 15) != 0);
        if (L > 0 && tid > 0 && vs < nv) mark_at = (int)vs;
      } else {
        const int64_t pn = l.pos[e + 1];
        if (pn > p && tid > 0 && vs < nv) mark_at = (int)vs;
        BlockPtrs ptrs;
        ptrs.sadj = sp - rel;
        ptrs.dadj = nullptr;
        s_sd[tid] = ptrs;
        s_careful[tid] = (sp - 15 < sbase || sp + (pn - p) + 16 > sbase + extent_of(a, sb)) ? 1 : 0;
      }
    }
    // vectors of the chunk this batch covers; a batch of empty blocks has none
    const int64_t first_rel = l.pos[b] - cA, next_rel = l.pos[b + cnt] - cA;
    const int vlo = first_rel > 0 ? (int)(first_rel >> 4) : 0;
    const int vhi = (next_rel >> 4) < nv ? (int)(next_rel >> 4) : nv;
    __syncthreads();
    if (vhi <= vlo) {
      // Nothing of this batch lies in the chunk.  If its blocks are all empty, the run
      // of empty blocks may go on for millions of descriptors (ranks that send or
      // receive nothing): stream positions do not move along it, so its end is found
      // by doubling steps and a bisection instead of batch by batch.  Every thread
      // reads the same entries and takes the same steps.
      if (next_rel == first_rel && b + cnt <= e_hi) {
        const int64_t p0 = first_rel + cA;
        int64_t lo = b + cnt, hi = lo, step = kBatch;  // pos[lo] == p0
        bool more = true;
        for (;;) {
          hi = lo + step < e_hi + 1 ? lo + step : e_hi + 1;  // (pos has an entry behind the last descriptor)
          if (l.pos[hi] > p0) break;
          if (hi == e_hi + 1) {
            more = false;  // empty to the end of this chunk's descriptors
            break;
          }
          lo = hi;
          step <<= 1;
        }
        if (!more) break;
        while (hi - lo > 1) {  // pos[lo] == p0 < pos[hi]
          const int64_t mid = lo + ((hi - lo) >> 1);
          if (l.pos[mid] > p0) hi = mid; else lo = mid;
        }
        b = lo - kBatch;  // descriptor lo is the first one with bytes: the next batch starts there
      }
      continue;
    }
    if (!waited) {  // everything above read only the plan's tables; the data may still be in the making
      grid_dependency_wait();
      waited = true;
    }
    const bool single = cnt == 1;
    if (single) {
      // One block covers the whole range (a chunk inside a large block).  If both
      // ends are 16-byte aligned and no vector of the range is partial, this is a
      // plain strided copy: no table look-ups in the loop.
      const char *src = s_sd[0].sadj + ((int64_t)vlo << 4);
      char *dst = (DELIVER ? s_sd[0].dadj : keep_out) + ((int64_t)vlo << 4);
      bool plain = (reinterpret_cast<uintptr_t>(src) & 15) == 0 && s_careful[0] == 0;
      if (DELIVER) plain = plain && s_oe[0].x <= (vlo << 4) && s_oe[0].y >= (vhi << 4);
      if (kBulk && a.bulk_off > 0 && plain && ((vhi - vlo) << 4) >= kBulkMin && ((vhi - vlo) << 4) <= kBulkBytes) {
        if (tid == 0) {
          const unsigned bytes = (unsigned)(vhi - vlo) << 4;
          const int np = (int)((bytes + kBulkPiece - 1) / kBulkPiece);
          char *stage = reinterpret_cast<char *>(s_who) + a.bulk_off;
          if (!bar_ready) {
            for (int j = 0; j < kBulkPieces; j++) mbar_init(smem_u32(&s_bar[j]), 1);
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
          }
          for (int j = 0; j < np; j++) {
            const unsigned off = (unsigned)j * kBulkPiece;
            const unsigned sz = bytes - off < (unsigned)kBulkPiece ? bytes - off : (unsigned)kBulkPiece;
            mbar_expect_tx(smem_u32(&s_bar[j]), sz);
            bulk_load(smem_u32(stage + off), src + off, sz, smem_u32(&s_bar[j]));
          }
          bool ok = true;
          for (int j = 0; j < np; j++) {
            const unsigned off = (unsigned)j * kBulkPiece;
            const unsigned sz = bytes - off < (unsigned)kBulkPiece ? bytes - off : (unsigned)kBulkPiece;
            if (ok && !mbar_wait(smem_u32(&s_bar[j]), (bulk_phase >> j) & 1)) ok = false;
            if (ok) {
              bulk_store(dst + off, smem_u32(stage + off), sz);
              bulk_commit();
            } else {
              (void)mbar_wait(smem_u32(&s_bar[j]), (bulk_phase >> j) & 1);  // one more bounded wait for the copy in flight
            }
          }
          bulk_wait_all();
          if (!ok) {
            if (a.error) atomicExch(a.error, 1);
            s_abort = 1;
          }
        }
        bar_ready = true;
        bulk_phase ^= (1u << ((((vhi - vlo) << 4) + kBulkPiece - 1) / kBulkPiece)) - 1;  // the barriers used
        continue;
      }
      if (plain) {
        const int m = vhi - vlo;
        int i = tid;
        for (; i + (kUnroll - 1) * kThreads < m; i += kUnroll * kThreads) {
          uint4 x[kUnroll];
#pragma unroll
          for (int k = 0; k < kUnroll; k++) x[k] = ld16(src + ((int64_t)(i + k * kThreads) << 4));
#pragma unroll
          for (int k = 0; k < kUnroll; k++) st16(dst + ((int64_t)(i + k * kThreads) << 4), x[k]);
        }
        for (; i < m; i += kThreads) st16(dst + ((int64_t)i << 4), ld16(src + ((int64_t)i << 4)));
        continue;
      }
      // The same range with a skewed source: still one block, every vector whole.
      // (Only in the build with registers to spare; lists of large blocks run it.)
      if constexpr (kUnroll >= 4) {
        bool whole = s_careful[0] == 0 && (reinterpret_cast<uintptr_t>(src) & 15) != 0;
        if (DELIVER) whole = whole && s_oe[0].x <= (vlo << 4) && s_oe[0].y >= (vhi << 4);
        if (whole) {
          skewed_run<kUnroll>(src, dst, vhi - vlo);
          continue;
        }
      }
    }
    if (!single) {
      if (mark_at >= 0) s_who[mark_at] = (unsigned char)tid;
      __syncthreads();
      fill_owner(s_who, s_vs, cnt, vlo, vhi);
      __syncthreads();
    }
    // every thread takes a strided share of the vectors: a few loads, then as many stores
    for (int v = vlo + tid; v - lane < vhi; v += kUnroll * kThreads) {  // whole warps stay in the loop
      uint4 x[kUnroll];
      char *out[kUnroll];
#pragma unroll
      for (int k = 0; k < kUnroll; k++) {
        const int vv = v + k * kThreads;
        bool on = vv < vhi;
        const char *sa = nullptr;
        bool careful = false;
        int t = 0, b0 = 0, b1 = 16;
        out[k] = nullptr;
        if (on) {
          if (!single) t = s_who[vv];
          const int64_t vb = (int64_t)vv << 4;
          const BlockPtrs ptrs = s_sd[t];
          if (DELIVER) {
            // A vector that lies wholly inside the block goes straight to its place.
            // The block's partial first and last vector are loaded here too, beside
            // their neighbours (the same cache lines), and parked in the block's two
            // slots of shared memory; the block's own thread stores their bytes later.
            const int2 oe = s_oe[t];
            const int org = oe.x, end = oe.y;
            b0 = org - (int)vb;
            b1 = end - (int)vb;
            const bool full = b0 <= 0 && b1 >= 16;
            on = b0 < 16 && b1 > 0;
            out[k] = full ? ptrs.dadj + vb
                          : reinterpret_cast<char *>(s_edge) + t * 32 + (b0 >= 0 ? 0 : 16);  // (b0 >= 0: the vector that holds the block's first byte)
          } else {
            out[k] = keep_out + vb;
          }
          sa = ptrs.sadj + vb;
          careful = s_careful[t] != 0;
          if (!on) out[k] = nullptr;
        }
        const bool aligned = (reinterpret_cast<uintptr_t>(sa) & 15) == 0;
        if (!l.skewed && __all_sync(0xffffffffu, !on || (aligned && !careful))) {
          if (on) x[k] = ld16(sa);
        } else if (on) {
          if (!careful) {
            x[k] = load16_pair(sa);
          } else if (DELIVER) {
            x[k] = load16_bytes(sa, b0 > 0 ? b0 : 0, b1 < 16 ? b1 : 16);
          } else {
            const int64_t e = b + t;
            const int64_t rem = l.len[e] - (cA + ((int64_t)vv << 4) - l.pos[e]);
            x[k] = load16_bytes(sa, 0, rem < 16 ? (int)(rem > 0 ? rem : 0) : 16);
          }
        }
      }
#pragma unroll
      for (int k = 0; k < kUnroll; k++)
        if (out[k]) st16(out[k], x[k]);  // (a generic store: global memory or the parking slot)
    }
    // DELIVER: the partial first and last vector of a block, by the block's own
    // thread, out of the parking slots
    if (DELIVER) {
      __syncthreads();
      if (my_edges) {
        const int vh = my_org >> 4, vt = (my_end - 1) >> 4;
        if (vh >= vlo && vh < vhi && ((my_org & 15) != 0 || my_end < (vh << 4) + 16)) {
          const int b0 = my_org - (vh << 4);
          const int b1 = my_end - (vh << 4) < 16 ? my_end - (vh << 4) : 16;
          store_pieces(s_sd[tid].dadj + ((int64_t)vh << 4), s_edge + tid * 32, b0, b1);
        }
        if (vt > vh && vt >= vlo && vt < vhi && (my_end & 15) != 0)
          store_pieces(s_sd[tid].dadj + ((int64_t)vt << 4), s_edge + tid * 32 + 16, 0, my_end - (vt << 4));
      }
    }
  }
}

// One launch, up to three lists: the block index picks the list and the chunk.
template <int kUnroll, bool kBulk>
__device__ __forceinline__ void launch_body(const TunaMoveArgs &a) {
  grid_launch_dependents();
  if (a.wait_first) grid_dependency_wait();  // the tables read below may be the previous kernel's output
  int64_t c = blockIdx.x;
  if (c < a.keep.nchunks) {
    move_body<false, kUnroll, kBulk>(a.keep, a, c);
  } else {
    c -= a.keep.nchunks;
    if (c < a.del.nchunks)
      move_body<true, kUnroll, kBulk>(a.del, a, c);
    else
      move_body<true, kUnroll, kBulk>(a.rot, a, c - a.del.nchunks);
  }
  // A CTA that found nothing to move has not waited yet.  Every CTA does before it
  // leaves, so that this launch cannot complete before its predecessor has, and the
  // next launch's wait covers the whole chain.
  grid_dependency_wait();
}

// Two builds of every kernel.  Lists of large blocks (from about 64 KiB) run best
// with four vectors in flight per thread and the registers that takes (4 CTAs per
// SM).  With smaller blocks a CTA spends much of its life on the dependent loads
// of its set-up (chunk table, descriptors, then data), so eight resident CTAs per
// SM with two vectors in flight each do better (measured: 1.15-1.4x on 180-byte
// blocks, 1.02x on 16 KiB blocks, 0.98x on 128 KiB blocks).
__global__ void __launch_bounds__(kThreads, 4) tuna_round_kernel(const TunaMoveArgs a) { launch_body<4, true>(a); }
__global__ void __launch_bounds__(kThreads, 4) tuna_rotate_kernel(const TunaMoveArgs a) { launch_body<4, true>(a); }
__global__ void __launch_bounds__(kThreads, 4) tuna_direct_kernel(const TunaMoveArgs a) { launch_body<4, true>(a); }
__global__ void __launch_bounds__(kThreads, 8) tuna_round_small_kernel(const TunaMoveArgs a) { launch_body<2, false>(a); }
__global__ void __launch_bounds__(kThreads, 8) tuna_rotate_small_kernel(const TunaMoveArgs a) { launch_body<2, false>(a); }
__global__ void __launch_bounds__(kThreads, 8) tuna_direct_small_kernel(const TunaMoveArgs a) { launch_body<2, false>(a); }

}  // namespace

cudaError_t tuna_launch_move(int kernel, const TunaMoveArgs &a_in, bool small_blocks, bool early_start,
                             cudaStream_t stream) {
  TunaMoveArgs a = a_in;
  const TunaListArgs *ls[3] = {&a.keep, &a.del, &a.rot};
  int64_t nchunks = 0, max_chunk = 0;
  for (const TunaListArgs *l : ls) {
    if (l->nchunks <= 0) continue;
    if (l->chunk > TUNA_MAX_CHUNK_BYTES || (l->chunk & 15)) return cudaErrorInvalidValue;
    nchunks += l->nchunks;
    max_chunk = l->chunk > max_chunk ? l->chunk : max_chunk;
  }
  if (nchunks <= 0) return cudaSuccess;
  const dim3 grid((unsigned)nchunks), block(kThreads);
  size_t who_bytes = (size_t)(max_chunk >> 4) + 32;  // one owner byte per 16-byte vector of a chunk (<= 16 KiB)
  const bool bulk = a.bulk_off != 0 && !small_blocks;  // the caller asks for the bulk-copy route
  a.bulk_off = 0;
  if (bulk) {  // the bulk staging area follows the owner table
    a.bulk_off = (int)((who_bytes + 127) & ~(size_t)127);
    who_bytes = a.bulk_off + kBulkBytes;
    // opt in to more than 48 KiB of dynamic shared memory, once per device
    static bool raised[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || !raised[dev]) {
      e = cudaFuncSetAttribute(tuna_round_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
      if (e == cudaSuccess) e = cudaFuncSetAttribute(tuna_rotate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
      if (e == cudaSuccess) e = cudaFuncSetAttribute(tuna_direct_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
      if (e != cudaSuccess) return e;
      if (dev >= 0 && dev < 64) raised[dev] = true;
    }
  }
  void (*fn)(const TunaMoveArgs);
  switch (kernel) {
    case TUNA_K_ROUND:
      fn = small_blocks ? tuna_round_small_kernel : tuna_round_kernel;
      break;
    case TUNA_K_ROTATE:
      fn = small_blocks ? tuna_rotate_small_kernel : tuna_rotate_kernel;
      break;
    default:
      fn = small_blocks ? tuna_direct_small_kernel : tuna_direct_kernel;
      break;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = who_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  static const bool chain = []() {  // TUNA_DEPENDENT_LAUNCH=0 turns the early start off
    const char *e = getenv("TUNA_DEPENDENT_LAUNCH");
    return !(e && e[0] == '0');
  }();
  cfg.attrs = attr;
  cfg.numAttrs = chain ? 1 : 0;
  a.wait_first = early_start ? 0 : 1;
  const cudaError_t le = cudaLaunchKernelEx(&cfg, fn, a);
  if (le != cudaSuccess) return le;
  return cudaGetLastError();
}
