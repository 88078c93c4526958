// The hierarchical exchange with its groups spread over several GPUs (Sec. IV of the
// paper: local rounds where bandwidth is high, one inter-group step across the slower
// link): group n of l ranks lives on GPU n.  Every GPU runs this library in a process of
// its own and builds the plan of its own share from the same, all-gathered count matrix:
//   local phases   radix-r rounds among the GPU's own l ranks, for all g destination
//                  groups at once, in the GPU's own memory (the same lists and the same
//                  mover as on one GPU, restricted to the ranks that live here);
//   global phase   the coalesced inter-group exchange (Sec. IV-B, Algorithm 3: g - 1
//                  rounds of one super-block each) as a PUSH: the sending GPU's mover
//                  reads every block where the local phases left it and stores it
//                  straight into its place in the receiving GPU's receive buffer, through
//                  a pointer the caller obtained by mapping that buffer into this process
//                  (plain 16-byte stores over NVLink; no cluster multicast, no bulk-copy
//                  route, and no library kernel is handed a peer pointer).
// Nothing here waits on another GPU: no flag, no spin, no device-side barrier.  The
// caller closes the exchange with a stream-ordered barrier across the GPUs (for
// instance an all-reduce enqueued behind this call on every GPU's stream); a GPU's
// receive buffer is complete when that barrier has passed.
#include <string.h>

#include "tuna_plan.h"

using namespace tuna_host;

extern "C" {

int tuna_shard_layout(int P, int n_gpus, int elem_size, const int64_t *sendcounts, const int64_t *sdispls,
                      const int64_t *rdispls, const int64_t *sendbase, const int64_t *recvbase,
                      int64_t *sendbase_out, int64_t *recvbase_out, int64_t *send_bytes,
                      int64_t *recv_bytes) {
  if (P < 1 || elem_size < 1 || n_gpus < 1 || !sendcounts) return TUNA_ERR_INVALID_ARG;
  if (P > TUNA_MAX_P) return TUNA_ERR_RANGE;
  if (P % n_gpus != 0) return TUNA_ERR_BAD_HIERARCHY;
  const int rc = validate_layout(P, sendcounts, sdispls, rdispls, sendbase, recvbase);
  if (rc) return rc;
  std::vector<int64_t> sb, rb, se, re;
  shard_layout(P, P / n_gpus, sendcounts, sdispls, rdispls, sendbase, recvbase, &sb, &rb, &se, &re);
  for (int p = 0; p < P; p++) {
    if (sendbase_out) sendbase_out[p] = sb[p];
    if (recvbase_out) recvbase_out[p] = rb[p];
  }
  for (int n = 0; n < n_gpus; n++) {
    if (send_bytes) send_bytes[n] = se[n] * elem_size;
    if (recv_bytes) recv_bytes[n] = re[n] * elem_size;
  }
  return TUNA_OK;
}

int tuna_shard_round_table(int P, int n_gpus, int my_gpu, int radix, int elem_size,
                           const int64_t *sendcounts, int cap, int *level, int *x, int *z,
                           int64_t *units, int64_t *bytes, int *rounds) {
  if (P < 1 || elem_size < 1 || n_gpus < 1 || !sendcounts || cap < 0) return TUNA_ERR_INVALID_ARG;
  if (P > TUNA_MAX_P) return TUNA_ERR_RANGE;
  if (P % n_gpus != 0) return TUNA_ERR_BAD_HIERARCHY;
  if (my_gpu < 0 || my_gpu >= n_gpus) return TUNA_ERR_INVALID_ARG;
  const int l = P / n_gpus, g = n_gpus;
  if (radix == 0) radix = std::max(2, l);
  if (radix < 2 || radix > std::max(2, l)) return TUNA_ERR_BAD_RADIX;
  for (int64_t i = 0; i < (int64_t)P * P; i++)
    if (sendcounts[i] < 0) return TUNA_ERR_INVALID_ARG;
  // Every block moves once per non-zero digit of its local offset (Sec. III-A, inside
  // the group) and once more if it leaves the group (Sec. IV-B, coalesced: round z
  // carries the super-blocks for the group z places on).  A round's bytes on this GPU:
  // the blocks its own ranks send in it.
  int k = 0;
  auto emit = [&](int lv, int xx, int zz, int64_t u, int64_t b) {
    if (k < cap) {
      if (level) level[k] = lv;
      if (x) x[k] = xx;
      if (z) z[k] = zz;
      if (units) units[k] = u;
      if (bytes) bytes[k] = b;
    }
    k++;
  };
  int64_t stride = 1;
  for (int xx = 0; stride < l; xx++, stride *= radix) {
    for (int zz = 1; zz < radix; zz++) {
      if ((int64_t)zz * stride >= l) continue;
      int64_t u = 0, b = 0;
      for (int q = 0; q < l; q++) {
        const int s = my_gpu * l + q;
        for (int d = 0; d < P; d++) {
          const int jo = ((d % l) - q + l) % l;
          if ((jo / stride) % radix != zz) continue;
          u++;
          b += sendcounts[(int64_t)s * P + d];
        }
      }
      emit(0, xx, zz, u, b * elem_size);
    }
  }
  for (int zz = 1; zz < g; zz++) {
    int64_t b = 0;
    const int dest = (my_gpu + zz) % g;
    for (int q = 0; q < l; q++)
      for (int j = 0; j < l; j++) b += sendcounts[(int64_t)(my_gpu * l + q) * P + dest * l + j];
    emit(1, 0, zz, l, b * elem_size);  // every rank of this GPU sends one super-block
  }
  if (rounds) *rounds = k;
  return TUNA_OK;
}

int tuna_shard_enable_peer_access(int peer_device) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    (void)cudaGetLastError();
    return TUNA_ERR_CUDA;
  }
  if (peer_device == dev) return TUNA_OK;
  int can = 0;
  if (cudaDeviceCanAccessPeer(&can, dev, peer_device) != cudaSuccess) {
    (void)cudaGetLastError();
    return TUNA_ERR_CUDA;
  }
  if (!can) return TUNA_ERR_INVALID_ARG;
  const cudaError_t e = cudaDeviceEnablePeerAccess(peer_device, 0);
  if (e != cudaSuccess) (void)cudaGetLastError();
  return (e == cudaSuccess || e == cudaErrorPeerAccessAlreadyEnabled) ? TUNA_OK : TUNA_ERR_CUDA;
}

int tuna_shard_plan_create(tuna_plan_t **out, int P, int radix, int n_gpus, int my_gpu, int elem_size,
                           unsigned flags, const int64_t *sendcounts, const int64_t *sdispls,
                           const int64_t *rdispls, const int64_t *sendbase, const int64_t *recvbase,
                           void *stream) {
  if (out) *out = nullptr;
  if (n_gpus < 1 || P < 1 || P % n_gpus != 0) return out ? TUNA_ERR_BAD_HIERARCHY : TUNA_ERR_INVALID_ARG;
  if (my_gpu < 0 || my_gpu >= n_gpus) return TUNA_ERR_INVALID_ARG;
  return plan_create(out, P, radix, 0, 0, P / n_gpus, n_gpus, elem_size, flags, sendcounts, sdispls, rdispls,
                     sendbase, recvbase, stream, n_gpus, my_gpu);
}

int tuna_shard_extents(const tuna_plan_t *pl, int gpu, size_t *send_bytes, size_t *recv_bytes) {
  if (!pl || pl->topo.shard_n == 0) return TUNA_ERR_INVALID_ARG;
  if (gpu < 0 || gpu >= pl->topo.shard_n) return TUNA_ERR_RANGE;
  if (send_bytes) *send_bytes = (size_t)pl->shard_send_extent[gpu];
  if (recv_bytes) *recv_bytes = (size_t)pl->shard_recv_extent[gpu];
  return TUNA_OK;
}

int tuna_shard_alltoallv(tuna_plan_t *pl, const void *sendbuf, void *const *recvbufs, int phases,
                         void *stream) {
  if (!pl || pl->topo.shard_n == 0 || !recvbufs) return TUNA_ERR_INVALID_ARG;
  if ((phases & ~(TUNA_SHARD_LOCAL | TUNA_SHARD_GLOBAL)) != 0 || phases == 0) return TUNA_ERR_INVALID_ARG;
  if (!pl->tables_valid) return TUNA_ERR_INTERNAL;
  const int N = pl->topo.shard_n, me = pl->topo.shard_me;
  if (!sendbuf && pl->send_extent > 0) return TUNA_ERR_INVALID_ARG;
  for (int n = 0; n < N; n++)
    if (!recvbufs[n] && pl->shard_recv_extent[n] > 0) return TUNA_ERR_INVALID_ARG;
  if (ranges_overlap(sendbuf, (size_t)pl->send_extent, recvbufs[me], (size_t)pl->recv_extent))
    return TUNA_ERR_OVERLAP;
  if (pl->workspace_need > 0 && (!pl->workspace || pl->workspace_bytes < (size_t)pl->workspace_need))
    return TUNA_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  {
    const int arc = await_tables(pl, st);
    if (arc) return arc;
  }
  // the GPUs' receive buffers as the mover looks them up (uploaded when they change;
  // the source is the plan's own host copy, which outlives the asynchronous copy)
  bool same = (int)pl->h_peer_ptrs.size() == N;
  for (int n = 0; same && n < N; n++) same = pl->h_peer_ptrs[n] == (char *)recvbufs[n];
  if (!same) {
    {
      const int wrc = wait_in_flight(pl);  // an exchange still running reads the table rewritten below
      if (wrc) return wrc;
    }
    pl->tables_fresh = true;  // (the launch that follows reads the table uploaded here)
    pl->h_peer_ptrs.assign(N, nullptr);
    for (int n = 0; n < N; n++) pl->h_peer_ptrs[n] = (char *)recvbufs[n];
    TUNA_CUDA(pl, cudaMemcpyAsync(pl->d_peer_ptrs, pl->h_peer_ptrs.data(), (size_t)N * sizeof(char *),
                                  cudaMemcpyHostToDevice, st));
  }
  int launches = 0, smalls = 0;
  bool rot_done = pl->rot.nchunks == 0 || !(phases & TUNA_SHARD_LOCAL);  // the self blocks belong to the local part
  for (size_t f = 0; f < pl->phases.size(); f++) {
    const int level = pl->phases[f].level;
    if (!(phases & (level == 0 ? TUNA_SHARD_LOCAL : TUNA_SHARD_GLOBAL))) continue;
    const TunaList &k = pl->keep[f];
    const TunaList &d = pl->deliver[f];
    const bool with_rot = !rot_done;
    if (k.nchunks == 0 && d.nchunks == 0 && !with_rot) continue;
    TunaMoveArgs a = move_args(pl, sendbuf, recvbufs[me], pl->workspace);
    a.bulk_off = 0;  // (the bulk-copy route is never taken towards another GPU's memory)
    a.keep = list_args(k);
    a.del = list_args(d);
    a.keep_base = pl->h_wbase[f];
    int64_t bytes = k.bytes + d.bytes;
    int64_t small_bytes = (k.small_blocks ? k.bytes : 0) + (d.small_blocks ? d.bytes : 0);
    if (with_rot) {
      a.rot = list_args(pl->rot);
      bytes += pl->rot.bytes;
      small_bytes += pl->rot.small_blocks ? pl->rot.bytes : 0;
      rot_done = true;
    }
    const bool small = 2 * small_bytes >= bytes;
    Timed tm(pl, level == 0 ? TUNA_TIMER_ROUND_LOCAL : TUNA_TIMER_ROUND_GLOBAL, bytes, st);
    TUNA_CUDA(pl, tuna_launch_move(TUNA_K_ROUND, a, small, launches > 0 || !pl->tables_fresh, st));
    launches++;
    smalls += small ? 1 : 0;
  }
  if (!rot_done) {  // no local phase had anything to carry them (one rank per GPU)
    Timed tm(pl, TUNA_TIMER_ROTATE, pl->rot.bytes, st);
    TunaMoveArgs a = move_args(pl, sendbuf, recvbufs[me], pl->workspace);
    a.bulk_off = 0;
    a.rot = list_args(pl->rot);
    TUNA_CUDA(pl, tuna_launch_move(TUNA_K_ROTATE, a, pl->rot.small_blocks, launches > 0 || !pl->tables_fresh, st));
    launches++;
    smalls += pl->rot.small_blocks ? 1 : 0;
  }
  pl->last_launches = launches;
  pl->last_small = smalls;
  pl->launch_count += launches;
  if (launches > 0) pl->tables_fresh = false;
  return launches > 0 ? mark_in_flight(pl, st) : TUNA_OK;
}

}  // extern "C"
