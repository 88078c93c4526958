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
//   tuna_round_kernel    KEEP lists.  The stream IS the destination, so stores
//                        are contiguous aligned vectors; sources are aligned
//                        workspace blocks or arbitrarily aligned send-buffer
//                        blocks (read as aligned words merged by funnel shifts).
//   tuna_deliver_kernel, tuna_rotate_kernel, tuna_direct_kernel
//                        DELIVER lists.  A vector whose destination is aligned and
//                        whole goes straight to global memory.  Everything else
//                        is gathered into shared memory at the destination's
//                        alignment and written out after a barrier: whole
//                        vectors with 16-byte stores, the partial first and last
//                        vector of a block in the widest aligned pieces that fit.
//                        No byte outside a block's destination range is written.
// No byte outside a source buffer's extent is read: blocks within 19 bytes of
// either end of their buffer are read byte by byte instead of by aligned windows.
#include "tuna_internal.h"

namespace {

constexpr int kThreads = TUNA_MOVE_THREADS;
constexpr int kBatch = kThreads;        // descriptors handled per batch (one per thread)
constexpr int kKeepVec = 4096;          // vectors per chunk of a KEEP list, at most (64 KiB)
constexpr int kKeepSpan = kKeepVec / kThreads;
constexpr int kStageVec = 2048;         // vectors of the staging window of a DELIVER list (32 KiB)
constexpr int kStageSpan = kStageVec / kThreads;
constexpr int kClampVec = 1 << 26;      // |vector index| beyond which only "far away" matters

__device__ __forceinline__ uint4 ld16(const char *p) { return *reinterpret_cast<const uint4 *>(p); }
__device__ __forceinline__ void st16(char *p, uint4 v) { *reinterpret_cast<uint4 *>(p) = v; }

// (a select, not an index: indexing a kernel parameter array spills it to local memory)
__device__ __forceinline__ char *base_of(const TunaMoveArgs &a, int buf) {
  return buf == TUNA_BUF_SEND ? a.base[0] : (buf == TUNA_BUF_RECV ? a.base[1] : a.base[2]);
}
__device__ __forceinline__ int64_t extent_of(const TunaMoveArgs &a, int buf) {
  return buf == TUNA_BUF_SEND ? a.extent[0] : (buf == TUNA_BUF_RECV ? a.extent[1] : a.extent[2]);
}

// Largest t < cnt with start[t] <= v (start is non-decreasing, start[0] <= v).
__device__ __forceinline__ int find_entry(const int *start, int cnt, int v) {
  int lo = 0;
#pragma unroll
  for (int step = kBatch / 2; step > 0; step >>= 1)
    if (lo + step < cnt && start[lo + step] <= v) lo += step;
  return lo;
}

// Owner table: who[v - v_first] = the descriptor owning vector v, for the vectors
// [v_first, v_last) of the current batch.  Each thread resolves SPAN consecutive
// vectors: one binary search for its last vector, then a walk down.
template <int SPAN>
__device__ __forceinline__ void fill_owner(unsigned char *who, const int *start, int cnt,
                                           int v_first, int v_last) {
  const int v0 = v_first + (int)threadIdx.x * SPAN;
  if (v0 >= v_last) return;
  const int vend = (v0 + SPAN < v_last) ? v0 + SPAN : v_last;
  int t = find_entry(start, cnt, vend - 1);
  for (int v = vend - 1; v >= v0; v--) {
    while (start[t] > v) t--;
    who[v - v_first] = (unsigned char)t;
  }
}

// The 16 bytes at sa (any alignment) from five aligned words merged by funnel shifts.
// Reads [sa - (sa & 3), +20).
__device__ __forceinline__ uint4 load16_funnel(const char *sa) {
  const unsigned sh = (unsigned)(reinterpret_cast<uintptr_t>(sa) & 3);
  const uint32_t *w = reinterpret_cast<const uint32_t *>(sa - sh);
  const uint32_t w0 = w[0], w1 = w[1], w2 = w[2], w3 = w[3], w4 = w[4];
  const unsigned bits = sh * 8;
  uint4 v;
  v.x = __funnelshift_r(w0, w1, bits);
  v.y = __funnelshift_r(w1, w2, bits);
  v.z = __funnelshift_r(w2, w3, bits);
  v.w = __funnelshift_r(w3, w4, bits);
  return v;
}

// Only the bytes [b0, b1) of the vector at sa, one by one (for blocks at the very
// ends of their source buffer, where an aligned window would leave it).
__device__ __noinline__ uint4 load16_bytes(const char *sa, int b0, int b1) {
  uint32_t w[4] = {0, 0, 0, 0};
  for (int i = b0; i < b1; i++) w[i >> 2] |= (uint32_t)(unsigned char)sa[i] << (8 * (i & 3));
  return make_uint4(w[0], w[1], w[2], w[3]);
}

// Store bytes [b0, b1) of the 16-byte vector at shared address sp to the 16-byte
// aligned global address gp, in the widest naturally aligned pieces that fit.
__device__ __forceinline__ void store_pieces(char *gp, const char *sp, int b0, int b1) {
  int pos = b0;
  while (pos < b1) {
    if (!(pos & 7) && pos + 8 <= b1) {
      *reinterpret_cast<uint2 *>(gp + pos) = *reinterpret_cast<const uint2 *>(sp + pos);
      pos += 8;
    } else if (!(pos & 3) && pos + 4 <= b1) {
      *reinterpret_cast<uint32_t *>(gp + pos) = *reinterpret_cast<const uint32_t *>(sp + pos);
      pos += 4;
    } else if (!(pos & 1) && pos + 2 <= b1) {
      *reinterpret_cast<unsigned short *>(gp + pos) = *reinterpret_cast<const unsigned short *>(sp + pos);
      pos += 2;
    } else {
      gp[pos] = sp[pos];
      pos += 1;
    }
  }
}

// ------------------------------------------------------------------ KEEP lists

__device__ __forceinline__ void keep_body(const TunaMoveArgs &a) {
  __shared__ int s_vs[kBatch];             // first vector of the block, relative to the chunk
  __shared__ const char *s_sadj[kBatch];   // source address of chunk vector v is s_sadj + 16 v
  __shared__ unsigned char s_careful[kBatch];
  __shared__ __align__(16) unsigned char s_who[kKeepVec];

  const int tid = threadIdx.x, lane = tid & 31;
  const int64_t c = blockIdx.x;
  const int64_t cA = c * a.chunk;
  const int64_t cB = (cA + a.chunk < a.total) ? cA + a.chunk : a.total;
  const int nv = (int)((cB - cA) >> 4);
  const int64_t e_lo = a.chunk_first[c];
  const int64_t e_hi = (c + 1 < a.nchunks) ? (int64_t)a.chunk_first[c + 1] : a.n - 1;
  char *const out = a.base[2] + a.keep_base + cA;

  for (int64_t b = e_lo; b <= e_hi; b += kBatch) {
    const int cnt = (int)((e_hi - b + 1 < kBatch) ? e_hi - b + 1 : kBatch);
    if (b > e_lo) __syncthreads();  // the previous batch is done with the tables
    if (tid < cnt) {
      const int64_t e = b + tid;
      const int64_t p = a.pos[e], pn = a.pos[e + 1];
      const int64_t s = a.src[e];
      const int sb = TUNA_LOC_BUF(s);
      const char *sbase = base_of(a, sb);
      const char *sp = sbase + TUNA_LOC_OFF(s);
      const int64_t rel = p - cA;
      int64_t vs = rel >> 4;
      if (vs < -kClampVec) vs = -kClampVec;
      s_vs[tid] = (int)vs;
      s_sadj[tid] = sp - rel;
      s_careful[tid] = (sp - 3 < sbase || sp + (pn - p) + 4 > sbase + extent_of(a, sb)) ? 1 : 0;
    }
    // vectors of the chunk this batch covers
    const int64_t first_rel = a.pos[b] - cA, next_rel = a.pos[b + cnt] - cA;
    const int vlo = first_rel > 0 ? (int)(first_rel >> 4) : 0;
    const int vhi = (next_rel >> 4) < nv ? (int)(next_rel >> 4) : nv;
    __syncthreads();
    const bool single = cnt == 1;
    if (!single) {
      fill_owner<kKeepSpan>(s_who, s_vs, cnt, vlo, vhi);
      __syncthreads();
    }
    for (int v = vlo + tid; v - lane < vhi; v += 4 * kThreads) {  // whole warps stay in the loop
      uint4 x[4];
#pragma unroll
      for (int k = 0; k < 4; k++) {
        const int vv = v + k * kThreads;
        const bool on = vv < vhi;
        const char *sa = nullptr;
        bool careful = false;
        int t = 0;
        if (on) {
          if (!single) t = s_who[vv - vlo];
          sa = s_sadj[t] + ((int64_t)vv << 4);
          careful = s_careful[t] != 0;
        }
        const bool aligned = (reinterpret_cast<uintptr_t>(sa) & 15) == 0;
        if (__all_sync(0xffffffffu, !on || (aligned && !careful))) {
          if (on) x[k] = ld16(sa);
        } else if (on) {
          if (!careful) {
            x[k] = load16_funnel(sa);
          } else {
            const int64_t e = b + t;
            const int64_t rem = a.len[e] - (cA + ((int64_t)vv << 4) - a.pos[e]);
            x[k] = load16_bytes(sa, 0, rem < 16 ? (int)(rem > 0 ? rem : 0) : 16);
          }
        }
      }
#pragma unroll
      for (int k = 0; k < 4; k++) {
        const int vv = v + k * kThreads;
        if (vv < vhi) st16(out + ((int64_t)vv << 4), x[k]);
      }
    }
  }
}

// ------------------------------------------------------------------ DELIVER lists

__device__ __forceinline__ void deliver_body(const TunaMoveArgs &a) {
  __shared__ __align__(16) char s_buf[kStageVec * 16];
  __shared__ int s_vs[kBatch];             // first vector of the block, relative to the chunk
  __shared__ int s_org[kBatch];            // chunk-relative byte position of the block's first byte
  __shared__ int s_end[kBatch];            // ... and one past its last byte (clamped when far away)
  __shared__ const char *s_sadj[kBatch];   // source address of chunk vector v is s_sadj + 16 v
  __shared__ char *s_dadj[kBatch];         // destination address likewise (16-byte aligned)
  __shared__ unsigned char s_careful[kBatch];
  __shared__ __align__(16) unsigned char s_who[kStageVec];

  const int tid = threadIdx.x, lane = tid & 31;
  const int64_t c = blockIdx.x;
  const int64_t cA = c * a.chunk;
  const int64_t cB = (cA + a.chunk < a.total) ? cA + a.chunk : a.total;
  const int nv = (int)((cB - cA) >> 4);
  const int64_t e_lo = a.chunk_first[c];
  const int64_t e_hi = (c + 1 < a.nchunks) ? (int64_t)a.chunk_first[c + 1] : a.n - 1;

  for (int64_t b = e_lo; b <= e_hi; b += kBatch) {
    const int cnt = (int)((e_hi - b + 1 < kBatch) ? e_hi - b + 1 : kBatch);
    if (b > e_lo) __syncthreads();  // the previous batch is done with the tables
    bool my_stage = false;
    int my_org = 0, my_end = 0;
    if (tid < cnt) {
      const int64_t e = b + tid;
      const int64_t p = a.pos[e];
      const int64_t L = a.len[e];
      const int64_t s = a.src[e], d = a.dst[e];
      const int sb = TUNA_LOC_BUF(s);
      const char *sbase = base_of(a, sb);
      const char *sp = sbase + TUNA_LOC_OFF(s);
      char *dp = base_of(a, TUNA_LOC_BUF(d)) + TUNA_LOC_OFF(d);
      const int ad = (int)(reinterpret_cast<uintptr_t>(dp) & 15);
      const int64_t rel = p - cA;
      int64_t vs = rel >> 4;
      if (vs < -kClampVec) vs = -kClampVec;
      const int64_t org = rel + ad;  // exact chunk-relative position of byte 0
      int64_t end = org + L;
      if (end > ((int64_t)kClampVec << 4)) end = (int64_t)kClampVec << 4;
      my_org = (int)(vs << 4) + ad;
      my_end = (int)end;
      s_vs[tid] = (int)vs;
      s_org[tid] = my_org;
      s_end[tid] = my_end;
      s_sadj[tid] = sp - org;
      s_dadj[tid] = dp - org;
      s_careful[tid] = (L > 0 && (sp - 19 < sbase || sp + L + 19 > sbase + extent_of(a, sb))) ? 1 : 0;
      my_stage = L > 0 && (ad != 0 || (L & 15) != 0);
    }
    const int64_t first_rel = a.pos[b] - cA, next_rel = a.pos[b + cnt] - cA;
    const int vlo = first_rel > 0 ? (int)(first_rel >> 4) : 0;
    const int vhi = (next_rel >> 4) < nv ? (int)(next_rel >> 4) : nv;
    const int any_stage = __syncthreads_or(my_stage ? 1 : 0);
    const bool single = cnt == 1;

    for (int w_lo = vlo; w_lo < vhi; w_lo += kStageVec) {
      const int w_hi = (w_lo + kStageVec < vhi) ? w_lo + kStageVec : vhi;
      if (w_lo > vlo) __syncthreads();  // the previous window is done with s_who and s_buf
      if (!single) {
        fill_owner<kStageSpan>(s_who, s_vs, cnt, w_lo, w_hi);
        __syncthreads();
      }
      // load a few vectors per thread, then store them: straight to global memory if
      // the destination is aligned and the vector whole, else into the staging buffer
      for (int v = w_lo + tid; v - lane < w_hi; v += 4 * kThreads) {  // whole warps stay in the loop
        uint4 x[4];
        char *out[4];
#pragma unroll
        for (int k = 0; k < 4; k++) {
          const int vv = v + k * kThreads;
          bool on = vv < w_hi;
          const char *sa = nullptr;
          bool careful = false;
          int b0 = 0, b1 = 16;
          out[k] = nullptr;
          if (on) {
            const int t = single ? 0 : s_who[vv - w_lo];
            const int org = s_org[t], end = s_end[t];
            const int vb = vv << 4;
            b0 = org - vb;
            b1 = end - vb;
            if (b1 <= 0) {
              on = false;  // the spare vector behind a block: nothing to move
            } else {
              sa = s_sadj[t] + (int64_t)vb;
              careful = s_careful[t] != 0;
              if ((org & 15) == 0 && b0 <= 0 && b1 >= 16) out[k] = s_dadj[t] + (int64_t)vb;
            }
          }
          const bool aligned = (reinterpret_cast<uintptr_t>(sa) & 15) == 0;
          if (__all_sync(0xffffffffu, !on || (aligned && !careful))) {
            if (on) x[k] = ld16(sa);
          } else if (on) {
            if (!careful)
              x[k] = load16_funnel(sa);
            else
              x[k] = load16_bytes(sa, b0 > 0 ? b0 : 0, b1 < 16 ? b1 : 16);
          }
          if (!on) out[k] = reinterpret_cast<char *>(1);  // marks "skip"
        }
#pragma unroll
        for (int k = 0; k < 4; k++) {
          const int vv = v + k * kThreads;
          if (out[k] == nullptr)
            *reinterpret_cast<uint4 *>(s_buf + ((vv - w_lo) << 4)) = x[k];
          else if (out[k] != reinterpret_cast<char *>(1))
            st16(out[k], x[k]);
        }
      }
      if (any_stage) {
        __syncthreads();
        // whole vectors of blocks with an unaligned destination
        for (int vv = w_lo + tid; vv < w_hi; vv += kThreads) {
          const int t = single ? 0 : s_who[vv - w_lo];
          const int org = s_org[t];
          if (org & 15) {
            const int vb = vv << 4;
            if (org <= vb && s_end[t] >= vb + 16)
              st16(s_dadj[t] + (int64_t)vb, *reinterpret_cast<const uint4 *>(s_buf + ((vv - w_lo) << 4)));
          }
        }
        // the partial first and last vector of a block: its own thread
        if (my_stage) {
          const int vh = my_org >> 4, vt = (my_end - 1) >> 4;
          if (vh >= w_lo && vh < w_hi && ((my_org & 15) != 0 || my_end < (vh << 4) + 16))
            store_pieces(s_dadj[tid] + ((int64_t)vh << 4), s_buf + ((vh - w_lo) << 4), my_org - (vh << 4),
                         my_end - (vh << 4) < 16 ? my_end - (vh << 4) : 16);
          if (vt > vh && vt >= w_lo && vt < w_hi && (my_end & 15) != 0)
            store_pieces(s_dadj[tid] + ((int64_t)vt << 4), s_buf + ((vt - w_lo) << 4), 0, my_end - (vt << 4));
        }
      }
    }
  }
}

__global__ void __launch_bounds__(kThreads) tuna_round_kernel(const TunaMoveArgs a) { keep_body(a); }
__global__ void __launch_bounds__(kThreads) tuna_deliver_kernel(const TunaMoveArgs a) { deliver_body(a); }
__global__ void __launch_bounds__(kThreads) tuna_rotate_kernel(const TunaMoveArgs a) { deliver_body(a); }
__global__ void __launch_bounds__(kThreads) tuna_direct_kernel(const TunaMoveArgs a) { deliver_body(a); }

}  // namespace

cudaError_t tuna_launch_move(int kernel, const TunaMoveArgs &a, cudaStream_t stream) {
  if (a.nchunks <= 0 || a.n <= 0) return cudaSuccess;
  const dim3 grid((unsigned)a.nchunks), block(kThreads);
  switch (kernel) {
    case TUNA_K_ROUND:
      if (a.chunk > (int64_t)kKeepVec * 16) return cudaErrorInvalidValue;
      tuna_round_kernel<<<grid, block, 0, stream>>>(a);
      break;
    case TUNA_K_DELIVER:
      tuna_deliver_kernel<<<grid, block, 0, stream>>>(a);
      break;
    case TUNA_K_ROTATE:
      tuna_rotate_kernel<<<grid, block, 0, stream>>>(a);
      break;
    default:
      tuna_direct_kernel<<<grid, block, 0, stream>>>(a);
      break;
  }
  return cudaGetLastError();
}
