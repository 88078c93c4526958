// The plan object and the host-side helpers shared by the translation units of the
// library (plan construction, exchange calls, the allocation-free entry point).
#ifndef TUNA_PLAN_H
#define TUNA_PLAN_H

#include <stdint.h>

#include <algorithm>
#include <vector>

#include "tuna_internal.h"

struct tuna_plan {
  TunaTopo topo{};
  int radix_l = 2, radix_g = 2;
  int block_count = 0;  // > 0: staggered inter-group exchange in batches of this many steps
  unsigned flags = 0;
  bool classic = false;
  int cuda_err = 0;
  int last_launches = 0;
  int last_small = 0;  // ... of which ran the small-block build of the mover

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
  // The tables have been rewritten since the last exchange was enqueued: the next exchange's first
  // launch must not read them before the kernels that wrote them are known to be complete.
  bool tables_fresh = true;
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

  // Sharded plan (topo.shard_n > 0): per GPU, the bytes of its send and receive buffer
  // the layout covers; on the device the receive extents (for the self-check) and the
  // GPUs' receive buffer addresses (for the mover), the latter set by every exchange call.
  std::vector<int64_t> shard_send_extent, shard_recv_extent;
  int64_t *d_peer_extent = nullptr;   // (a slice of d_readback, like the three below)
  int64_t *d_shard_send_total = nullptr, *d_shard_recv_total = nullptr, *d_shard_send_extent = nullptr;
  char **d_peer_ptrs = nullptr;
  std::vector<char *> h_peer_ptrs;  // what d_peer_ptrs was last given

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

constexpr int64_t kStaticSmallBlockBytes = 65536;  // the table-free entry point decides by size alone
constexpr int64_t kHostStagingBlockBytes = 2048;   // mean block below which host buffers are staged

namespace tuna_host {

int mark_in_flight(tuna_plan *pl, cudaStream_t st);
int wait_in_flight(tuna_plan *pl);
int mark_tables_ready(tuna_plan *pl, cudaStream_t st);
int await_tables(tuna_plan *pl, cudaStream_t st);
cudaEvent_t take_event(tuna_plan *pl);
int validate_layout(int P, const int64_t *counts, const int64_t *sdispls, const int64_t *rdispls,
                    const int64_t *sendbase, const int64_t *recvbase);
// Creates a plan; shard_n > 0 makes it the plan of GPU shard_me among shard_n (then
// g == shard_n, the global radix is g, and sendbase / recvbase are per GPU).
int plan_create(tuna_plan_t **out, int P, int radix, int radix_global, int block_count, int l, int g,
                int elem_size, unsigned flags, const int64_t *sendcounts, const int64_t *sdispls,
                const int64_t *rdispls, const int64_t *sendbase, const int64_t *recvbase, void *stream,
                int shard_n = 0, int shard_me = 0);
// Region bases of a sharded layout: every GPU's buffers hold the regions of its own l
// ranks; a NULL base array means they are packed in rank order from offset 0 of that
// GPU's buffer.  Also every GPU's buffer extents, in elements.
void shard_layout(int P, int l, const int64_t *counts, const int64_t *sdispls, const int64_t *rdispls,
                  const int64_t *sendbase, const int64_t *recvbase, std::vector<int64_t> *sb,
                  std::vector<int64_t> *rb, std::vector<int64_t> *send_extent,
                  std::vector<int64_t> *recv_extent);
TunaListArgs list_args(const TunaList &l);
TunaMoveArgs move_args(const tuna_plan *pl, const void *send, void *recv, char *work);
// Multiprocessors of the current device (read once per device; 148 on a B200).
int sm_count();

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

template <class T>
cudaError_t dev_alloc(T **p, int64_t n) {
  return cudaMalloc((void **)p, (size_t)std::max<int64_t>(n, 1) * sizeof(T));
}

inline bool ranges_overlap(const void *a, size_t na, const void *b, size_t nb) {
  const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
  return na > 0 && nb > 0 && a0 < b0 + nb && b0 < a0 + na;
}

inline int64_t align256(int64_t v) { return (v + 255) & ~(int64_t)255; }

}  // namespace tuna_host

#endif
