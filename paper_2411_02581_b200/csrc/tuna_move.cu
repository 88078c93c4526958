// Fused pack-move-unpack kernels.
//
// One launch executes every copy descriptor of one list: a digit phase of the
// radix-r schedule (all rounds z of one digit position x: the blocks whose x-th
// offset digit equals z leave the rank that holds them and land, already in
// their slot order, in the buffer of the rank at distance +z*r^x; Sec. III-A/B of
// the paper), the final rotation into the MPI_Alltoallv receive layout, or the
// single-pass direct exchange (Sec. II-d).  "Pack" is the gather from the
// source rank's buffer, "move" the rank shift, "unpack" the placement at the
// destination offset; with all ranks in one memory the three are one copy, so
// each payload byte is read once and written once per hop.
//
// Work is partitioned by bytes, not by blocks: the destination stream of a list
// (blocks in receive-side order, each padded to 16 bytes) is cut into equal
// chunks, one CTA per chunk, and a precomputed table gives the first descriptor
// of every chunk.  A block larger than a chunk is therefore spread over several
// CTAs, and a chunk of tiny blocks is shared out over the threads of one CTA.
//
// Inside a CTA every piece of a block takes one of two routes:
//   direct  - source and destination both 16-byte aligned and the piece is large:
//             the pieces are laid end to end as one run of 16-byte vectors and
//             every thread copies a strided share of that run, four loads in
//             flight before the first store.
//   staged  - small pieces and pieces whose two ends are aligned differently: all
//             of them are gathered into shared memory first (every thread again
//             takes a strided share of the vectors, whatever block they belong
//             to), placed so that the shared-memory address is congruent to the
//             destination address modulo 16; after a barrier the same vectors
//             are written out with aligned 16-byte stores, partial ones at the
//             two ends of a block with the widest aligned stores that fit.  No
//             byte outside a block's destination range is written, and no byte
//             outside the source buffer's extent is read.
#include "tuna_internal.h"

namespace {

constexpr int kThreads = TUNA_MOVE_THREADS;
constexpr int kWarps = kThreads / 32;
constexpr int kBatch = kThreads;      // descriptors handled per batch (one per thread)
constexpr int kStage = 32768;         // bytes of staging buffer
constexpr int kStageVec = kStage / 16;
constexpr int kDirectMin = 4096;      // aligned pieces at least this long skip the staging buffer

__device__ __forceinline__ uint4 ld16(const char *p) { return *reinterpret_cast<const uint4 *>(p); }
__device__ __forceinline__ void st16(char *p, uint4 v) { *reinterpret_cast<uint4 *>(p) = v; }

// (a select, not an index: indexing a kernel parameter array spills it to local memory)
__device__ __forceinline__ char *base_of(const TunaMoveArgs &a, int buf) {
  return buf == TUNA_BUF_SEND ? a.base[0] : (buf == TUNA_BUF_RECV ? a.base[1] : a.base[2]);
}

// Largest t < cnt with start[t] <= v (start is non-decreasing, start[0] <= v).
__device__ __forceinline__ int find_entry(const int *start, int cnt, int v) {
  int lo = 0;
#pragma unroll
  for (int step = kBatch / 2; step > 0; step >>= 1)
    if (lo + step < cnt && start[lo + step] <= v) lo += step;
  return lo;
}

// Exclusive prefix sum over the CTA (one value per thread); *total gets the sum.
__device__ __forceinline__ int block_exclusive_scan(int x, int *s_warp, int *total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = x;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += y;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  int woff = 0, tot = 0;
#pragma unroll
  for (int k = 0; k < kWarps; k++) {
    const int w = s_warp[k];
    if (k < warp) woff += w;
    tot += w;
  }
  *total = tot;
  __syncthreads();
  return woff + incl - x;
}

// The 16 source bytes starting at sa (any alignment), read with aligned accesses.
// [lo, hi) is the extent of the buffer sa points into; if the aligned window would
// leave it, only the bytes [b0, b1) of the vector are read, one by one.
__device__ __forceinline__ uint4 load16_any(const char *sa, const char *lo, const char *hi, int b0,
                                            int b1) {
  const unsigned r = (unsigned)(reinterpret_cast<uintptr_t>(sa) & 15);
  uint4 v;
  if (r == 0) {
    if (sa >= lo && sa + 16 <= hi) return ld16(sa);
  } else if ((r & 3) == 0) {
    if (sa >= lo && sa + 16 <= hi) {
      const uint32_t *w = reinterpret_cast<const uint32_t *>(sa);
      v.x = w[0];
      v.y = w[1];
      v.z = w[2];
      v.w = w[3];
      return v;
    }
  } else {
    const unsigned sh = r & 3;
    const char *wb = sa - sh;
    if (wb >= lo && wb + 20 <= hi) {
      const uint32_t *w = reinterpret_cast<const uint32_t *>(wb);
      const uint32_t w0 = w[0], w1 = w[1], w2 = w[2], w3 = w[3], w4 = w[4];
      const unsigned bits = sh * 8;
      v.x = __funnelshift_r(w0, w1, bits);
      v.y = __funnelshift_r(w1, w2, bits);
      v.z = __funnelshift_r(w2, w3, bits);
      v.w = __funnelshift_r(w3, w4, bits);
      return v;
    }
  }
  // at the very edge of the buffer: only the bytes that belong to the block
  unsigned char b[16];
#pragma unroll
  for (int i = 0; i < 16; i++) b[i] = (i >= b0 && i < b1) ? (unsigned char)sa[i] : 0;
  v.x = b[0] | (b[1] << 8) | (b[2] << 16) | ((unsigned)b[3] << 24);
  v.y = b[4] | (b[5] << 8) | (b[6] << 16) | ((unsigned)b[7] << 24);
  v.z = b[8] | (b[9] << 8) | (b[10] << 16) | ((unsigned)b[11] << 24);
  v.w = b[12] | (b[13] << 8) | (b[14] << 16) | ((unsigned)b[15] << 24);
  return v;
}

// Store bytes [b0, b1) of the vector v to the 16-byte aligned address p, using the
// widest naturally aligned stores that stay inside the range.
__device__ __forceinline__ void store16_partial(char *p, uint4 v, int b0, int b1) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int q = 0; q < 2; q++) {  // the two 8-byte halves
    const int h0 = q * 8;
    if (b0 <= h0 && b1 >= h0 + 8) {
      *reinterpret_cast<uint2 *>(p + h0) = make_uint2(w[2 * q], w[2 * q + 1]);
      continue;
    }
#pragma unroll
    for (int k = 0; k < 2; k++) {  // the 4-byte words of this half
      const int w0 = h0 + k * 4;
      const uint32_t x = w[2 * q + k];
      if (b0 <= w0 && b1 >= w0 + 4) {
        *reinterpret_cast<uint32_t *>(p + w0) = x;
        continue;
      }
#pragma unroll
      for (int j = 0; j < 2; j++) {  // the 2-byte halves of this word
        const int s0 = w0 + j * 2;
        const uint32_t y = (x >> (16 * j)) & 0xffffu;
        if (b0 <= s0 && b1 >= s0 + 2) {
          *reinterpret_cast<unsigned short *>(p + s0) = (unsigned short)y;
        } else {
          if (b0 <= s0 && b1 > s0) p[s0] = (char)(y & 0xff);
          if (b0 <= s0 + 1 && b1 > s0 + 1) p[s0 + 1] = (char)(y >> 8);
        }
      }
    }
  }
}

__device__ __forceinline__ void move_body(const TunaMoveArgs &a) {
  __shared__ __align__(16) char s_buf[kStage];
  __shared__ const char *s_src[kBatch];
  __shared__ char *s_dst[kBatch];
  __shared__ int s_n[kBatch];         // clipped length of the piece in bytes
  __shared__ int s_dvec[kBatch];      // direct route: first vector of the piece in the run
  __shared__ int s_svec[kBatch];      // staged route: first vector of the piece in the staging stream
  __shared__ unsigned char s_who[kStageVec];  // staged route: piece that owns each staged vector
  __shared__ int s_warp[kWarps];

  const int tid = threadIdx.x;
  const int64_t c = blockIdx.x;
  const int64_t lo_pos = c * a.chunk;
  const int64_t hi_pos = (lo_pos + a.chunk < a.total) ? lo_pos + a.chunk : a.total;
  const int64_t e_lo = a.chunk_first[c];
  const int64_t e_hi = (c + 1 < a.nchunks) ? (int64_t)a.chunk_first[c + 1] : a.n - 1;

  for (int64_t b = e_lo; b <= e_hi; b += kBatch) {
    const int cnt = (int)((e_hi - b + 1 < kBatch) ? e_hi - b + 1 : kBatch);
    // ---- one descriptor per thread: clip to the chunk, classify ----
    int n = 0, dvec = 0, svec = 0;
    bool src_is_send = false, dst_is_work = false;
    const char *src = nullptr;
    char *dst = nullptr;
    if (tid < cnt) {
      const int64_t e = b + tid;
      const int64_t p0 = a.pos[e];
      const int64_t L = a.len[e];
      const int64_t lo = (p0 > lo_pos ? p0 : lo_pos) - p0;
      const int64_t hi = (p0 + L < hi_pos ? p0 + L : hi_pos) - p0;
      if (hi > lo) {
        n = (int)(hi - lo);
        const int64_t s = a.src[e], d = a.dst[e];
        src = base_of(a, TUNA_LOC_BUF(s)) + TUNA_LOC_OFF(s) + lo;
        dst = base_of(a, TUNA_LOC_BUF(d)) + TUNA_LOC_OFF(d) + lo;
        src_is_send = TUNA_LOC_BUF(s) == TUNA_BUF_SEND;
        dst_is_work = TUNA_LOC_BUF(d) == TUNA_BUF_WORK;
        const unsigned al = (unsigned)((reinterpret_cast<uintptr_t>(src) | reinterpret_cast<uintptr_t>(dst)) & 15);
        if (al == 0 && n >= kDirectMin)
          dvec = n >> 4;  // whole vectors go direct; a ragged tail (< 16 bytes) is staged
      }
    }
    const int a_dst = (int)(reinterpret_cast<uintptr_t>(dst) & 15);
    // what is left for the staging route: everything, or only the ragged tail
    int stage_n = n, stage_skip = 0;
    if (dvec > 0) {
      stage_skip = dvec << 4;
      stage_n = n - stage_skip;
    }
    if (stage_n > 0) svec = (stage_n + a_dst + 15) >> 4;
    int dtotal, stotal;
    const int dstart = block_exclusive_scan(dvec, s_warp, &dtotal);
    const int sstart = block_exclusive_scan(svec, s_warp, &stotal);
    s_src[tid] = src;
    s_dst[tid] = dst;
    // flags packed beside the length: bit 30 = destination is the workspace,
    // bit 29 = source is the send buffer; lengths are below 2^29 by construction
    s_n[tid] = n | (dst_is_work ? (1 << 30) : 0) | (src_is_send ? (1 << 29) : 0);
    s_dvec[tid] = dstart;
    s_svec[tid] = sstart;
    __syncthreads();

    // ---- direct route: one run of aligned vectors ----
    if (dtotal > 0) {
      int v = tid;
      for (; v + 3 * kThreads < dtotal; v += 4 * kThreads) {
        uint4 x[4];
        char *out[4];
#pragma unroll
        for (int k = 0; k < 4; k++) {
          const int vv = v + k * kThreads;
          const int t = find_entry(s_dvec, cnt, vv);
          const int64_t off = (int64_t)(vv - s_dvec[t]) << 4;
          x[k] = ld16(s_src[t] + off);
          out[k] = s_dst[t] + off;
        }
#pragma unroll
        for (int k = 0; k < 4; k++) st16(out[k], x[k]);
      }
      for (; v < dtotal; v += kThreads) {
        const int t = find_entry(s_dvec, cnt, v);
        const int64_t off = (int64_t)(v - s_dvec[t]) << 4;
        st16(s_dst[t] + off, ld16(s_src[t] + off));
      }
    }

    // ---- staged route, one window of the staging stream at a time ----
    for (int w0 = 0; w0 < stotal; w0 += kStageVec) {
      const int wn = (stotal - w0 < kStageVec) ? stotal - w0 : kStageVec;
      if (w0 > 0) __syncthreads();  // the previous window has been written out
      // gather
      for (int v = tid; v < wn; v += 4 * kThreads) {
        uint4 x[4];
#pragma unroll
        for (int k = 0; k < 4; k++) {
          const int vv = v + k * kThreads;
          if (vv < wn) {
            const int g = w0 + vv;
            const int t = find_entry(s_svec, cnt, g);
            const int nn = s_n[t];
            const int len = nn & ((1 << 29) - 1);
            const bool whole_direct = false;
            (void)whole_direct;
            const char *sp = s_src[t];
            const int ad = (int)(reinterpret_cast<uintptr_t>(s_dst[t]) & 15);
            // bytes of the piece that go through staging start at `skip`
            const int dv = (t + 1 < cnt ? s_dvec[t + 1] : dtotal) - s_dvec[t];
            const int skip = dv << 4;
            const int off = ((g - s_svec[t]) << 4) - ad;  // first byte of this vector, relative to skip
            const int b0 = off < 0 ? -off : 0;
            const int rem = (len - skip) - off;
            const int b1 = rem < 16 ? rem : 16;
            const char *sa = sp + skip + off;
            const bool from_send = (nn >> 29) & 1;
            const char *elo = from_send ? a.base[0] : a.base[2];
            const char *ehi = elo + (from_send ? a.extent[0] : a.extent[2]);
            x[k] = load16_any(sa, elo, ehi, b0, b1);
            s_who[vv] = (unsigned char)t;
          }
        }
#pragma unroll
        for (int k = 0; k < 4; k++) {
          const int vv = v + k * kThreads;
          if (vv < wn) *reinterpret_cast<uint4 *>(s_buf + (vv << 4)) = x[k];
        }
      }
      __syncthreads();
      // scatter
      for (int vv = tid; vv < wn; vv += kThreads) {
        const int g = w0 + vv;
        const int t = s_who[vv];
        const int nn = s_n[t];
        const int len = nn & ((1 << 29) - 1);
        char *dp = s_dst[t];
        const int ad = (int)(reinterpret_cast<uintptr_t>(dp) & 15);
        const int dv = (t + 1 < cnt ? s_dvec[t + 1] : dtotal) - s_dvec[t];
        const int skip = dv << 4;
        const int off = ((g - s_svec[t]) << 4) - ad;
        const int b0 = off < 0 ? -off : 0;
        const int rem = (len - skip) - off;
        const int b1 = rem < 16 ? rem : 16;
        const uint4 x = *reinterpret_cast<const uint4 *>(s_buf + (vv << 4));
        char *da = dp + skip + off;
        if ((b0 == 0 && b1 == 16) || ((nn >> 30) & 1))
          st16(da, x);  // whole vector, or padding of our own workspace
        else
          store16_partial(da, x, b0, b1);
      }
    }
    __syncthreads();  // shared tables are rewritten by the next batch
  }
}

__global__ void __launch_bounds__(kThreads) tuna_round_kernel(const TunaMoveArgs a) { move_body(a); }
__global__ void __launch_bounds__(kThreads) tuna_rotate_kernel(const TunaMoveArgs a) { move_body(a); }
__global__ void __launch_bounds__(kThreads) tuna_direct_kernel(const TunaMoveArgs a) { move_body(a); }

}  // namespace

cudaError_t tuna_launch_move(int kind, const TunaMoveArgs &a, cudaStream_t stream) {
  if (a.nchunks <= 0 || a.n <= 0) return cudaSuccess;
  const dim3 grid((unsigned)a.nchunks), block(kThreads);
  switch (kind) {
    case TUNA_MOVE_ROUND:
      tuna_round_kernel<<<grid, block, 0, stream>>>(a);
      break;
    case TUNA_MOVE_ROTATE:
      tuna_rotate_kernel<<<grid, block, 0, stream>>>(a);
      break;
    default:
      tuna_direct_kernel<<<grid, block, 0, stream>>>(a);
      break;
  }
  return cudaGetLastError();
}
