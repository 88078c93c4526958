// The direct exchange for callers that must not allocate device memory: every
// table in one file-scope device array.
#include <mutex>

#include "tuna_plan.h"
#include "tuna_plan_kernels.cuh"

using namespace tuna_host;

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
  // Sizes first, with every product and sum kept far from overflow: an entry so large
  // that bytes, displacement + count or base + region could wrap is refused here,
  // before anything is added up, and so is a work stream above the limit; both
  // before the buffers are looked at, so that nothing is ever launched for them.
  const int64_t kMaxElems = (INT64_MAX >> 16) / elem_size;  // 2^47 bytes: no sum of 2 P + 1 such terms wraps
  for (int64_t i = 0; i < PP; i++) {
    if (sendcounts[i] > kMaxElems || (sdispls && sdispls[i] > kMaxElems) || (rdispls && rdispls[i] > kMaxElems))
      return TUNA_ERR_RANGE;
  }
  for (int p = 0; p < P; p++)
    if ((sendbase && sendbase[p] > kMaxElems) || (recvbase && recvbase[p] > kMaxElems)) return TUNA_ERR_RANGE;
  const int64_t kMaxStream = (int64_t)TUNA_STATIC_MAX_CHUNKS * TUNA_MAX_CHUNK_BYTES;  // 4 GiB
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
      if (stream_bytes > kMaxStream) return TUNA_ERR_RANGE;  // (also keeps the running sums small)
      if (sdispls) sreg[s] = std::max(sreg[s], sdispls[(int64_t)s * P + d] + c); else sreg[s] += c;
      if (rdispls) rreg[d] = std::max(rreg[d], rdispls[(int64_t)d * P + s] + c); else rreg[d] += c;
    }
  int64_t se = 0, re = 0, acc_s = 0, acc_r = 0;
  for (int p = 0; p < P; p++) {
    sb[p] = sendbase ? sendbase[p] : acc_s;
    rb[p] = recvbase ? recvbase[p] : acc_r;
    acc_s += sreg[p];
    acc_r += rreg[p];
    if (sb[p] + sreg[p] > kMaxElems || rb[p] + rreg[p] > kMaxElems) return TUNA_ERR_RANGE;
    se = std::max(se, sb[p] + sreg[p]);
    re = std::max(re, rb[p] + rreg[p]);
  }
  se *= elem_size;
  re *= elem_size;
  int64_t chunk = 8192;
  while (chunk < TUNA_MAX_CHUNK_BYTES &&
         ((chunk < 65536 && stream_bytes / chunk > sm_count() * 32) ||
          (stream_bytes + chunk - 1) / chunk > TUNA_STATIC_MAX_CHUNKS))
    chunk <<= 1;
  const int64_t nchunks = (stream_bytes + chunk - 1) / chunk;
  if (nchunks > TUNA_STATIC_MAX_CHUNKS) return TUNA_ERR_RANGE;  // more than 4 GiB of work stream
  if ((!sendbuf && se > 0) || (!recvbuf && re > 0)) return TUNA_ERR_INVALID_ARG;
  if (ranges_overlap(sendbuf, (size_t)se, recvbuf, (size_t)re)) return TUNA_ERR_OVERLAP;
  if (payload == 0) return TUNA_OK;
  cudaStream_t st = (cudaStream_t)stream;
  {
    // The uploads below hand host arrays (the caller's and this frame's) to
    // asynchronous copies.  Issued eagerly the runtime stages them before it returns;
    // recorded into a graph they would be read again, from memory long gone, at every
    // replay.  So a stream that is being captured is refused.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) {
      (void)cudaGetLastError();
      return TUNA_ERR_CUDA;
    }
    if (cap != cudaStreamCaptureStatusNone) return TUNA_ERR_INVALID_ARG;
  }

  StaticTables t;
  if (static_tables(&t) != cudaSuccess) return TUNA_ERR_CUDA;
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
  TUNA_STATIC_CUDA(tuna_launch_move(TUNA_K_DIRECT, a, payload / PP < kStaticSmallBlockBytes, false, st));
#undef TUNA_STATIC_CUDA
  return TUNA_OK;
}

}  // extern "C"
