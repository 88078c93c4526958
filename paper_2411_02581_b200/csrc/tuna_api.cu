// C-ABI entry points that run an exchange or report on a plan.
#include <string.h>

#include "tuna_plan.h"

namespace tuna_host {

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
  a.skewed = 2 * l.unaligned_bytes > l.bytes ? 1 : 0;
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
  a.peer = pl->d_peer_ptrs;
  a.error = pl->d_error;
  a.bulk_off = (pl->flags & TUNA_FLAG_BULK_COPY) ? 1 : 0;
  return a;
}

}  // namespace tuna_host

using namespace tuna_host;

namespace {

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
  int launches = 0, smalls = 0;
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
    TUNA_CUDA(pl, tuna_launch_move(TUNA_K_ROUND, a, small, launches > 0 || !pl->tables_fresh, st));
    launches++;
    smalls += small ? 1 : 0;
  }
  if (!rot_done) {
    Timed tm(pl, TUNA_TIMER_ROTATE, pl->rot.bytes, st);
    TunaMoveArgs a = move_args(pl, send, recv, pl->workspace);
    a.rot = list_args(pl->rot);
    TUNA_CUDA(pl, tuna_launch_move(TUNA_K_ROTATE, a, pl->rot.small_blocks, launches > 0 || !pl->tables_fresh, st));
    launches++;
    smalls += pl->rot.small_blocks ? 1 : 0;
  }
  pl->last_small = smalls;
  pl->last_launches = launches;
  pl->launch_count += launches;
  if (launches > 0) pl->tables_fresh = false;  // (a launch that waited in full has run behind the plan kernels)
  return launches > 0 ? mark_in_flight(pl, st) : TUNA_OK;
}

int run_direct(tuna_plan *pl, const void *send, void *recv, cudaStream_t st) {
  if (pl->no_direct) return TUNA_ERR_INVALID_ARG;  // the plan was created without a direct list
  {
    const int arc = await_tables(pl, st);
    if (arc) return arc;
  }
  int launches = 0;
  pl->last_small = 0;
  if (pl->dir_shared) {  // the single phase's DELIVER list and the self blocks: every block, once
    const TunaList &d = pl->deliver[0];
    if (d.nchunks > 0 || pl->rot.nchunks > 0) {
      const int64_t bytes = d.bytes + pl->rot.bytes;
      const int64_t small_bytes = (d.small_blocks ? d.bytes : 0) + (pl->rot.small_blocks ? pl->rot.bytes : 0);
      Timed tm(pl, TUNA_TIMER_DIRECT, bytes, st);
      TunaMoveArgs a = move_args(pl, send, recv, nullptr);
      a.del = list_args(d);
      a.rot = list_args(pl->rot);
      TUNA_CUDA(pl, tuna_launch_move(TUNA_K_DIRECT, a, 2 * small_bytes >= bytes, !pl->tables_fresh, st));
      launches++;
      pl->last_small = 2 * small_bytes >= bytes ? 1 : 0;
    }
  } else if (pl->dir.nchunks > 0) {
    Timed tm(pl, TUNA_TIMER_DIRECT, pl->dir.bytes, st);
    TunaMoveArgs a = move_args(pl, send, recv, nullptr);
    a.del = list_args(pl->dir);
    TUNA_CUDA(pl, tuna_launch_move(TUNA_K_DIRECT, a, pl->dir.small_blocks, !pl->tables_fresh, st));
    launches++;
    pl->last_small = pl->dir.small_blocks ? 1 : 0;
  }
  pl->last_launches = launches;
  pl->launch_count += launches;
  if (launches > 0) pl->tables_fresh = false;  // (a launch that waited in full has run behind the plan kernels)
  return launches > 0 ? mark_in_flight(pl, st) : TUNA_OK;
}

}  // namespace

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
  if (pl->topo.shard_n > 0) return TUNA_ERR_INVALID_ARG;  // a sharded plan runs through tuna_shard_alltoallv
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
  if (pl->topo.shard_n > 0) return TUNA_ERR_INVALID_ARG;  // a sharded plan runs through tuna_shard_alltoallv
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
  if (pl->topo.shard_n > 0) return TUNA_ERR_INVALID_ARG;  // a sharded plan runs through tuna_shard_alltoallv
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

int tuna_rows_alltoallv(tuna_plan_t *pl, const void *rows_in, void *rows_out, void *stream) {
  if (!pl) return TUNA_ERR_INVALID_ARG;
  if (pl->topo.shard_n > 0) return TUNA_ERR_INVALID_ARG;  // a sharded plan runs through tuna_shard_alltoallv
  if (!pl->rows_valid) return TUNA_ERR_COUNT_MISMATCH;
  const TunaList &l = pl->rowsl;
  if (l.n > 0 && (!rows_in || !rows_out)) return TUNA_ERR_INVALID_ARG;
  if (ranges_overlap(rows_in, (size_t)pl->rows_in_bytes, rows_out, (size_t)pl->rows_out_bytes))
    return TUNA_ERR_OVERLAP;
  int launches = 0;
  pl->last_small = 0;
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
    TUNA_CUDA(pl, tuna_launch_move(TUNA_K_DIRECT, a, l.small_blocks, !pl->tables_fresh, st));
    launches++;
    pl->last_small = l.small_blocks ? 1 : 0;
  }
  pl->last_launches = launches;
  pl->launch_count += launches;
  if (launches > 0) pl->tables_fresh = false;  // (a launch that waited in full has run behind the plan kernels)
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

int tuna_plan_last_small_launches(const tuna_plan_t *pl, int *launches) {
  if (!pl || !launches) return TUNA_ERR_INVALID_ARG;
  *launches = pl->last_small;
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

}  // extern "C"
