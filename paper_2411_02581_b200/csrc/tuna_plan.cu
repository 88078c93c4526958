// Plan construction and update: the host path that validates a layout, uploads it,
// runs the plan kernels (count-metadata exchange + segmented prefix sums, Sec. III-B/C
// of the paper) and reads back the few totals that size the workspace and the grids;
// with the C-ABI entry points that create, update and destroy a plan.
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

#include <atomic>
#include <condition_variable>
#include <functional>
#include <mutex>
#include <new>
#include <thread>

#include "tuna_plan.h"
#include "tuna_plan_kernels.cuh"

namespace tuna_host {

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

void shard_layout(int P, int l, const int64_t *counts, const int64_t *sdispls, const int64_t *rdispls,
                  const int64_t *sendbase, const int64_t *recvbase, std::vector<int64_t> *sb,
                  std::vector<int64_t> *rb, std::vector<int64_t> *send_extent,
                  std::vector<int64_t> *recv_extent) {
  const int g = P / l;
  std::vector<int64_t> sreg(P, 0), rreg(P, 0);  // elements every rank's regions span
  for (int s = 0; s < P; s++)
    for (int d = 0; d < P; d++) {
      const int64_t c = counts[(int64_t)s * P + d];
      if (sdispls) sreg[s] = std::max(sreg[s], sdispls[(int64_t)s * P + d] + c); else sreg[s] += c;
      if (rdispls) rreg[d] = std::max(rreg[d], rdispls[(int64_t)d * P + s] + c); else rreg[d] += c;
    }
  sb->assign(P, 0);
  rb->assign(P, 0);
  send_extent->assign(g, 0);
  recv_extent->assign(g, 0);
  for (int n = 0; n < g; n++) {
    int64_t acc_s = 0, acc_r = 0;  // packed: a GPU's regions back to back, from 0
    for (int q = 0; q < l; q++) {
      const int p = n * l + q;
      (*sb)[p] = sendbase ? sendbase[p] : acc_s;
      (*rb)[p] = recvbase ? recvbase[p] : acc_r;
      acc_s += sreg[p];
      acc_r += rreg[p];
      (*send_extent)[n] = std::max((*send_extent)[n], (*sb)[p] + sreg[p]);
      (*recv_extent)[n] = std::max((*recv_extent)[n], (*rb)[p] + rreg[p]);
    }
  }
}

int sm_count() {
  static int cached[64] = {};
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return 148;
  }
  if (dev >= 0 && dev < 64 && cached[dev] > 0) return cached[dev];
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
    (void)cudaGetLastError();
    return 148;
  }
  if (dev >= 0 && dev < 64) cached[dev] = n;
  return n;
}

}  // namespace tuna_host

using namespace tuna_host;

namespace {

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
  while (c < top && l.total / c > sm_count() * 32) c <<= 1;
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
      if (t.shard_n > 0) {  // this GPU's buffers; the self-check needs every GPU's receive extent
        pl->send_extent = pl->shard_send_extent[t.shard_me];
        pl->recv_extent = pl->shard_recv_extent[t.shard_me];
        TUNA_CUDA(pl, cudaMemcpyAsync(pl->d_peer_extent, pl->shard_recv_extent.data(), (size_t)t.shard_n * 8,
                                      cudaMemcpyHostToDevice, st));
      }
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
      if (!hl && t.shard_n > 0) {  // every GPU's send regions laid end to end from 0 of its own buffer
        tuna_shard_bases_kernel<<<(unsigned)((P + th - 1) / th), th, 0, st>>>(pl->d_seg_total, P, t.Q, pl->d_sendbase,
                                                                              pl->d_shard_send_total);
        TUNA_LAUNCHED(pl);
      } else if (!hl) {  // send regions laid end to end: bases = scan of the row sums
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
      if (!hl && t.shard_n > 0) {
        tuna_shard_bases_kernel<<<(unsigned)((P + th - 1) / th), th, 0, st>>>(pl->d_seg_total, P, t.Q, pl->d_recvbase,
                                                                              pl->d_shard_recv_total);
        TUNA_LAUNCHED(pl);
        tuna_shard_extents_kernel<<<1, 32, 0, st>>>(pl->d_shard_send_total, pl->d_shard_recv_total, t.shard_n,
                                                    t.shard_me, t.elem, pl->d_extents, pl->d_peer_extent,
                                                    pl->d_shard_send_extent);
        TUNA_LAUNCHED(pl);
      } else if (!hl) {  // receive regions likewise: scan of the column sums
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
    // (a plan that starts with a digit phase reads sizes and locations off the layout there)
    const bool init_tables = nph == 0 || pl->phases[0].stag_hi > 0;
    tuna_init_tables_kernel<<<gPP, th, 0, st>>>(t, pl->d_counts, pl->d_sdispls, pl->d_rdispls,
                                                pl->d_sendbase, pl->d_recvbase, init_tables ? pl->d_sz[0] : nullptr,
                                                init_tables ? pl->d_loc[0] : nullptr, pl->dir.len, pl->dir.src, pl->dir.dst,
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
      // (the tables that follow the blocks have no reader behind the last phase)
      int64_t *const sz_next = f + 1 < nph ? pl->d_sz[cur ^ 1] : nullptr;
      int64_t *const loc_next = f + 1 < nph ? pl->d_loc[cur ^ 1] : nullptr;
      const TunaFirst first = f == 0 ? TunaFirst{pl->d_counts, pl->d_sdispls, pl->d_sendbase}
                                     : TunaFirst{nullptr, nullptr, nullptr};
      if (ph.level == 0 && ph.stride == 1 && ph.radix >= t.Q && t.N <= 65535) {
        const unsigned tiles = (unsigned)((t.Q + 31) / 32);
        tuna_meta_exchange_diag_kernel<<<dim3(tiles * tiles, t.N, t.N), dim3(32, 8), 0, st>>>(
            t, pd, first, pl->d_sz[cur], pl->d_loc[cur], sz_next, k.len, k.src, d.len, d.src,
            pl->d_round_bytes + ph.stats_off);
      } else {
        const size_t smem = ph.radix <= 4096 ? (size_t)ph.radix * 8 : 0;
        tuna_meta_exchange_kernel<<<gPP, th, smem, st>>>(t, pd, first, pl->d_sz[cur], pl->d_loc[cur],
                                                         sz_next, k.len, k.src, d.len, d.src,
                                                         pl->d_round_bytes + ph.stats_off);
      }
      TUNA_LAUNCHED(pl);
      // per-rank prefix sums of both lists; the KEEP stream is this phase's workspace region
      rc = scan_phase_lists(pl, k, ph.per_rank - ph.finals, f, pl->d_wbase + f, d, ph.finals, nph + f, st);
      if (rc) return rc;
      tuna_place_kernel<<<gPP, th, 0, st>>>(t, pd, first, pl->d_loc[cur], loc_next, k.pos,
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
      const unsigned gx = (unsigned)std::min<int64_t>((pl->check_max_n + th - 1) / th, (int64_t)sm_count() * 8);
      tuna_check_lists_kernel<<<dim3(gx, pl->n_check_items), th, 0, st>>>(
          static_cast<const TunaCheckItem *>(pl->d_check_items), pl->d_extents, pl->d_wbase + nph, pl->d_wbase,
          pl->d_violations, pl->d_peer_extent);
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
    if (t.shard_n > 0) {  // every GPU's buffer sizes, worked out on the device
      std::vector<int64_t> both(2 * (size_t)t.shard_n);
      if (pl->h_readback) {
        const int64_t *h = pl->h_readback + (pl->d_shard_send_extent - pl->d_readback);
        std::copy(h, h + 2 * t.shard_n, both.begin());
      } else {
        TUNA_CUDA(pl, cudaMemcpy(both.data(), pl->d_shard_send_extent, both.size() * 8, cudaMemcpyDeviceToHost));
      }
      for (int n = 0; n < t.shard_n; n++) {
        pl->shard_send_extent[n] = both[n];
        pl->shard_recv_extent[n] = both[t.shard_n + n];
      }
    }
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
  pl->tables_fresh = true;
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

}  // namespace

extern "C" {

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
  cudaFree(pl->d_peer_ptrs);
  for (auto &s : pl->stamps) {
    cudaEventDestroy(s.a);
    cudaEventDestroy(s.b);
  }
  for (auto e : pl->event_pool) cudaEventDestroy(e);
  delete pl;
  return TUNA_OK;
}

}  // extern "C"

int tuna_host::plan_create(tuna_plan_t **out, int P, int radix, int radix_global, int block_count,
                           int l, int g, int elem_size, unsigned flags, const int64_t *sendcounts,
                           const int64_t *sdispls, const int64_t *rdispls, const int64_t *sendbase,
                           const int64_t *recvbase, void *stream, int shard_n, int shard_me) {
  if (!out) return TUNA_ERR_INVALID_ARG;
  *out = nullptr;
  if (P < 1 || elem_size < 1 || !sendcounts || l < 1 || g < 1) return TUNA_ERR_INVALID_ARG;
  if (P > TUNA_MAX_P) return TUNA_ERR_RANGE;
  if ((int64_t)l * g != P) return TUNA_ERR_BAD_HIERARCHY;
  if (shard_n > 0) {
    // one group per GPU, one hop between GPUs, blocks delivered straight into the receive
    // buffers, no direct list (a GPU reaches only its own send buffer)
    if (shard_n != g || shard_me < 0 || shard_me >= shard_n || block_count != 0 ||
        shard_n > TUNA_MAX_SHARDS || (flags & (TUNA_FLAG_CLASSIC_ROTATE | TUNA_FLAG_BULK_COPY)))
      return TUNA_ERR_INVALID_ARG;
    radix_global = std::max(2, g);
    flags |= TUNA_FLAG_NO_DIRECT;
  }
  // radix 0 = choose: one hop per level (with all ranks in one memory every further
  // hop only adds a read and a write of the block; there is no message latency to save)
  if (radix == 0) radix = std::max(2, l);
  if (radix_global == 0 && block_count == 0) radix_global = std::max(2, g);
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
  std::vector<int64_t> shard_sb, shard_rb;
  if (shard_n > 0) {  // region bases are per GPU: worked out here, explicit from here on
    int vrc = validate_layout(P, sendcounts, sdispls, rdispls, sendbase, recvbase);
    if (vrc) {
      tuna_plan_destroy(pl);
      return vrc;
    }
    shard_layout(P, l, sendcounts, sdispls, rdispls, sendbase, recvbase, &shard_sb, &shard_rb,
                 &pl->shard_send_extent, &pl->shard_recv_extent);
    for (auto &v : pl->shard_send_extent) v *= elem_size;
    for (auto &v : pl->shard_recv_extent) v *= elem_size;
    sendbase = shard_sb.data();
    recvbase = shard_rb.data();
  }
  int rc = host_layout(P, sendcounts, sdispls, rdispls, sendbase, recvbase, &hl, pl->h_buf[0]);
  if (rc) {
    tuna_plan_destroy(pl);
    return rc;
  }
  pl->h_cur = 0;
  pl->h_counts = pl->h_buf[0];
  pl->topo = TunaTopo{P, l, g, elem_size, shard_n, shard_me};
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
    const int64_t n_shard = 4 * (int64_t)shard_n;  // the GPUs' send and receive totals and extents
    pl->readback_words = n_scal + n_wbase + n_ext + n_rb + n_viol + n_shard;
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
    if (shard_n > 0) {
      pl->d_shard_send_total = reinterpret_cast<int64_t *>(pl->d_violations + n_viol);
      pl->d_shard_recv_total = pl->d_shard_send_total + shard_n;
      pl->d_shard_send_extent = pl->d_shard_recv_total + shard_n;
      pl->d_peer_extent = pl->d_shard_send_extent + shard_n;
    }
  }
  TUNA_TRY(dev_alloc(&pl->d_error, 1));
  if (shard_n > 0) {
    TUNA_TRY(dev_alloc(&pl->d_peer_ptrs, shard_n));
    TUNA_TRY(cudaMemset(pl->d_peer_ptrs, 0, (size_t)shard_n * sizeof(char *)));
  }
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

extern "C" {

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
  std::vector<int64_t> shard_sb, shard_rb, shard_se, shard_re;
  if (pl->topo.shard_n > 0) {  // a sharded plan's region bases are per GPU
    const int vrc = validate_layout(pl->topo.P, sendcounts, sdispls, rdispls, sendbase, recvbase);
    if (vrc) return vrc;
    shard_layout(pl->topo.P, pl->topo.Q, sendcounts, sdispls, rdispls, sendbase, recvbase, &shard_sb, &shard_rb,
                 &shard_se, &shard_re);
    sendbase = shard_sb.data();
    recvbase = shard_rb.data();
  }
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
  if (pl->topo.shard_n > 0) {
    for (int n = 0; n < pl->topo.shard_n; n++) {
      pl->shard_send_extent[n] = shard_se[n] * pl->topo.elem;
      pl->shard_recv_extent[n] = shard_re[n] * pl->topo.elem;
    }
  }
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

int tuna_plan_set_row_maps(tuna_plan_t *pl, const int64_t *gather_rows, const int64_t *scatter_rows,
                           int64_t in_rows, int64_t out_rows, void *stream) {
  if (!pl || in_rows < 0 || out_rows < 0 || pl->topo.shard_n > 0) return TUNA_ERR_INVALID_ARG;
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
    tuna_check_list_kernel<<<(unsigned)std::min<int64_t>((n + th - 1) / th, (int64_t)sm_count() * 8), th, 0, st>>>(
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
  pl->tables_fresh = true;
  return TUNA_OK;
}

}  // extern "C"
