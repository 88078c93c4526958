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
// CTAs, and a chunk of tiny blocks is shared out between the warps of one CTA.
#include "tuna_internal.h"

namespace {

constexpr int kThreads = TUNA_MOVE_THREADS;
constexpr int kWarps = kThreads / 32;
constexpr int kBatch = kThreads;       // descriptors staged in shared memory at a time
constexpr int kCtaWide = 4096;         // clipped length from which the whole CTA copies one block

__device__ __forceinline__ uint4 ld16(const char *p) {
  return *reinterpret_cast<const uint4 *>(p);
}
__device__ __forceinline__ void st16(char *p, uint4 v) { *reinterpret_cast<uint4 *>(p) = v; }

// n bytes, one byte per thread per step, by a group of G threads (t = id in group).
__device__ __forceinline__ void copy_bytes(char *dst, const char *src, int64_t n, int t, int G) {
  for (int64_t i = t; i < n; i += G) dst[i] = src[i];
}

// m 16-byte vectors, both sides 16-byte aligned.
template <int UNROLL>
__device__ __forceinline__ void copy_vec(char *dst, const char *src, int64_t m, int t, int G) {
  int64_t i = t;
  for (; i + (int64_t)(UNROLL - 1) * G < m; i += (int64_t)UNROLL * G) {
    uint4 v[UNROLL];
#pragma unroll
    for (int k = 0; k < UNROLL; k++) v[k] = ld16(src + (i + (int64_t)k * G) * 16);
#pragma unroll
    for (int k = 0; k < UNROLL; k++) st16(dst + (i + (int64_t)k * G) * 16, v[k]);
  }
  for (; i < m; i += G) st16(dst + i * 16, ld16(src + i * 16));
}

// Copy n bytes between arbitrary byte addresses, touching only bytes inside
// [src, src+n) and [dst, dst+n).  Stores are 16-byte vectors on the destination's
// alignment; the source is read as 16-byte vectors (co-aligned), 4-byte words
// (offset a multiple of 4) or pairs of aligned words merged by a funnel shift.
__device__ __forceinline__ void copy_any(char *dst, const char *src, int64_t n, int t, int G) {
  if (n <= 0) return;
  int64_t h = (16 - (reinterpret_cast<uintptr_t>(dst) & 15)) & 15;
  if (h > n) h = n;
  copy_bytes(dst, src, h, t, G);
  dst += h;
  src += h;
  n -= h;
  const int64_t m = n >> 4;
  const unsigned s = (unsigned)(reinterpret_cast<uintptr_t>(src) & 15);
  if (s == 0) {
    copy_vec<4>(dst, src, m, t, G);
  } else if ((s & 3) == 0) {
    for (int64_t i = t; i < m; i += G) {
      const uint32_t *w = reinterpret_cast<const uint32_t *>(src + i * 16);
      uint4 v;
      v.x = w[0];
      v.y = w[1];
      v.z = w[2];
      v.w = w[3];
      st16(dst + i * 16, v);
    }
  } else {
    // Vector i needs the 20 aligned bytes starting at src + 16 i - sh.  For the
    // first and the last vector that window pokes outside [src, src + 16 m), so
    // those two go byte by byte.
    const unsigned sh = s & 3;
    const unsigned bits = sh * 8;
    const uint32_t *base = reinterpret_cast<const uint32_t *>(src - sh);
    for (int64_t i = t + 1; i < m - 1; i += G) {
      const uint32_t *w = base + i * 4;
      const uint32_t w0 = w[0], w1 = w[1], w2 = w[2], w3 = w[3], w4 = w[4];
      uint4 v;
      v.x = __funnelshift_r(w0, w1, bits);
      v.y = __funnelshift_r(w1, w2, bits);
      v.z = __funnelshift_r(w2, w3, bits);
      v.w = __funnelshift_r(w3, w4, bits);
      st16(dst + i * 16, v);
    }
    if (m >= 1) copy_bytes(dst, src, 16, t, G);
    if (m >= 2) copy_bytes(dst + (m - 1) * 16, src + (m - 1) * 16, 16, t, G);
  }
  copy_bytes(dst + m * 16, src + m * 16, n & 15, t, G);
}

// (a select, not an index: indexing a kernel parameter array spills it to local memory)
__device__ __forceinline__ char *base_of(const TunaMoveArgs &a, int buf) {
  return buf == TUNA_BUF_SEND ? a.base[0] : (buf == TUNA_BUF_RECV ? a.base[1] : a.base[2]);
}

__device__ __forceinline__ void move_body(const TunaMoveArgs &a) {
  __shared__ const char *s_src[kBatch];
  __shared__ char *s_dst[kBatch];
  __shared__ int64_t s_n[kBatch];

  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  const int64_t c = blockIdx.x;
  const int64_t lo_pos = c * a.chunk;
  const int64_t hi_pos = (lo_pos + a.chunk < a.total) ? lo_pos + a.chunk : a.total;
  const int64_t e_lo = a.chunk_first[c];
  const int64_t e_hi = (c + 1 < a.nchunks) ? (int64_t)a.chunk_first[c + 1] : a.n - 1;

  for (int64_t b = e_lo; b <= e_hi; b += kBatch) {
    const int cnt = (int)((e_hi - b + 1 < kBatch) ? e_hi - b + 1 : kBatch);
    __syncthreads();
    if (tid < cnt) {
      const int64_t e = b + tid;
      const int64_t p0 = a.pos[e];
      const int64_t L = a.len[e];
      const int64_t lo = (p0 > lo_pos ? p0 : lo_pos) - p0;
      const int64_t hi = (p0 + L < hi_pos ? p0 + L : hi_pos) - p0;
      int64_t n = hi - lo;
      if (n > 0) {
        const int64_t s = a.src[e], d = a.dst[e];
        s_src[tid] = base_of(a, TUNA_LOC_BUF(s)) + TUNA_LOC_OFF(s) + lo;
        s_dst[tid] = base_of(a, TUNA_LOC_BUF(d)) + TUNA_LOC_OFF(d) + lo;
      } else {
        n = 0;
      }
      s_n[tid] = n;
    }
    __syncthreads();
    // large pieces: the whole CTA on one block at a time
    for (int i = 0; i < cnt; i++) {
      const int64_t n = s_n[i];
      if (n >= kCtaWide) copy_any(s_dst[i], s_src[i], n, tid, kThreads);
    }
    // the rest: one warp per block
    for (int i = warp; i < cnt; i += kWarps) {
      const int64_t n = s_n[i];
      if (n > 0 && n < kCtaWide) copy_any(s_dst[i], s_src[i], n, lane, 32);
    }
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
