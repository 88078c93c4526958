/*
 * tuna.h - C ABI of the TuNA (tunable-radix non-uniform all-to-all) library for
 * one NVIDIA B200.
 *
 * All P logical ranks live inside one GPU: the "send buffers" of the P ranks are
 * regions of a single device buffer, likewise the "receive buffers".  The exchange
 * has exactly the semantics of MPI_Alltoallv (the paper's Sec. VI-B and Conclusion
 * state that the algorithms keep its signature and meaning): block j of rank i's
 * send region arrives as block i of rank j's receive region; bytes of the receive
 * buffer that no block covers are left untouched.
 *
 * Conventions for every function
 *   - returns TUNA_OK (0) or a negative tuna_status; never aborts; a validation
 *     failure touches no GPU state.
 *   - "host" pointers are ordinary CPU memory, "device" pointers are CUDA device
 *     memory of the current device.  The library copies every host array it is
 *     given before returning; the caller may free them at once.
 *   - counts and displacements are 64-bit and in ELEMENTS of elem_size bytes.
 *     Matrices are row-major P x P: sendcounts[s*P + d], sdispls[s*P + d]
 *     (relative to rank s's send region), rdispls[d*P + s] (relative to rank d's
 *     receive region).  sendbase[p] / recvbase[p] give the element offset of rank
 *     p's region inside the one send / receive buffer.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *     Work is enqueued on it; unless stated otherwise nothing synchronises.
 *   - the caller owns send buffer, receive buffer and workspace; the plan owns
 *     only its descriptor tables, freed by tuna_plan_destroy.
 */
#ifndef TUNA_H
#define TUNA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tuna_plan tuna_plan_t;

#define TUNA_MAX_P 32768 /* ranks of one plan, at most */

typedef enum tuna_status {
  TUNA_OK = 0,
  TUNA_ERR_INVALID_ARG = -1,    /* null pointer, P < 1, elem_size < 1, negative count or offset */
  TUNA_ERR_BAD_RADIX = -2,      /* radix outside [2, max(2, ranks of its level)] */
  TUNA_ERR_BAD_HIERARCHY = -3,  /* l * g != P */
  TUNA_ERR_COUNT_MISMATCH = -4, /* counts/displacements differ from the plan's, or recv != send^T */
  TUNA_ERR_OVERLAP = -5,        /* send and receive ranges alias (no in-place exchange) */
  TUNA_ERR_WORKSPACE = -6,      /* workspace missing, misaligned or too small */
  TUNA_ERR_CUDA = -7,           /* a CUDA runtime call failed; see tuna_plan_cuda_error */
  TUNA_ERR_NOMEM = -8,          /* host or device allocation of the plan's tables failed */
  TUNA_ERR_RANGE = -9,          /* index (round, phase, ...) out of range, or size above a stated limit */
  TUNA_ERR_INTERNAL = -10       /* the plan's self-check failed: a descriptor would leave its buffers;
                                   nothing has been moved and the plan must not be used */
} tuna_status;

/* flags for tuna_plan_create */
#define TUNA_FLAG_DIRECT_TO_R 0u    /* default: a block's last hop writes straight into the receive buffer */
#define TUNA_FLAG_CLASSIC_ROTATE 1u /* last hops land in the workspace; one final rotation pass reorders them */
#define TUNA_FLAG_BULK_COPY 2u      /* chunks inside one large 16-byte aligned block go through the SM's bulk
                                       copy engine (cp.async.bulk through shared memory) instead of vector loads
                                       and stores; same result, measured about 1 % slower, hence optional */
#define TUNA_FLAG_NO_DIRECT 4u      /* the plan will not be used for tuna_direct_alltoallv (nor the direct schedule
                                       of tuna_alltoallv_host): no separate direct list is built, which shortens
                                       every update of a multi-phase plan; those calls return TUNA_ERR_INVALID_ARG */

/* schedules for the host-buffer entry point */
#define TUNA_SCHEDULE_TUNA 0
#define TUNA_SCHEDULE_DIRECT 1

/*
 * tuna_plan_create - build the schedule and every displacement for one count matrix.
 *
 * Defines: Sec. III-A (radix-r rounds: round (x, z) moves the blocks whose x-th
 * base-r digit of the offset (dst - src) mod P equals z to the rank at distance
 * +z*r^x), Sec. III-B (per-round metadata: the sizes of the blocks a rank holds,
 * obtained here by applying the same rank shift to the size table), Sec. III-C
 * (placement of intermediate blocks; here exact offsets from segmented exclusive
 * prefix sums over the sizes instead of max-size slots), Sec. IV (hierarchical
 * variant: ranks p = n*l + q; local rounds of radix `radix` on the local offset
 * inside every group of l consecutive ranks, for all g destination groups at
 * once; then global rounds of radix `radix_global` on the group offset between
 * ranks with equal local id; radix_global == g is the paper's coalesced exchange).
 *
 *   out           host; receives the plan.
 *   P             number of ranks, 1 <= P <= TUNA_MAX_P (TUNA_ERR_RANGE above: the
 *                 tables index P * P blocks with 32-bit arithmetic).
 *   radix         flat radix (g == 1) or local radix, in [2, max(2, l)], or 0 = choose.
 *   radix_global  global radix in [2, max(2, g)], or 0 = choose; ignored when g == 1.
 *                 The choice is the largest radix, l and g: one hop per level.  The
 *                 paper's Sec. V-A finds small radices best for small blocks, where
 *                 per-message latency dominates, and large ones for large blocks,
 *                 where the bytes forwarded dominate; with every rank in one memory
 *                 there is no per-message latency to save, only the forwarding cost
 *                 (each hop reads and writes the block once more), and every measured
 *                 workload ran fastest with the fewest hops.
 *   l, g          ranks per group and number of groups, l*g == P; g == 1 is flat TuNA.
 *   elem_size     bytes per element, >= 1.
 *   flags         TUNA_FLAG_*.
 *   sendcounts    host, P*P.
 *   sdispls, rdispls, sendbase, recvbase
 *                 host, P*P / P*P / P / P; any of them may be NULL, meaning blocks
 *                 packed back to back in ascending index order (sdispls, rdispls)
 *                 and regions packed in rank order (sendbase, recvbase); these
 *                 defaults are computed on the device by the same scan kernel.
 *   stream        the plan kernels run on it; the call synchronises it once to read
 *                 back the phase totals that size the workspace.
 * Before returning, a device-side self-check verifies that every descriptor of
 * every list reads inside [0, send_bytes) or the workspace and writes inside
 * [0, recv_bytes) or the workspace (TUNA_ERR_INTERNAL otherwise): the exchange
 * kernels touch only those ranges, so no exchange can access memory out of bounds.
 */
int tuna_plan_create(tuna_plan_t **out, int P, int radix, int radix_global, int l, int g,
                     int elem_size, unsigned flags, const int64_t *sendcounts,
                     const int64_t *sdispls, const int64_t *rdispls, const int64_t *sendbase,
                     const int64_t *recvbase, void *stream);

/*
 * tuna_plan_create_staggered - hierarchical plan whose inter-group phase is the
 * staggered exchange.
 *
 * Computes: the local phase of tuna_plan_create (Sec. IV-A), then Sec. IV-B's
 * staggered pattern as Algorithm 2 states it: a step index ii = gi*l + gr runs over
 * [0, P) in batches of `block_count`; in step (gi, gr), gi >= 1, rank (n, q) sends
 * the single block whose original owner is rank (n, gr) to rank ((n - gi) mod g, q)
 * and receives from rank ((n + gi) mod g, q) the block owned by ((n + gi) mod g, gr),
 * straight into the receive buffer.  Nothing is compacted into super-blocks.  The
 * steps of one batch share one kernel launch (the counterpart of the requests that
 * are in flight together), so the exchange takes one launch per local digit phase
 * plus one per batch that moves anything; block_count >= P gives a single batch.
 *
 *   block_count   steps per batch, >= 1.
 *   radix         local radix in [2, max(2, l)].
 *   flags         TUNA_FLAG_CLASSIC_ROTATE is not supported here (TUNA_ERR_INVALID_ARG).
 * All other arguments, ownership and errors as tuna_plan_create.  Every function
 * taking a plan accepts this one.  Its rounds of level 1 are the l*(g-1) steps in
 * order, reported by tuna_plan_round_info with x = gi, z = gr and units = P (one
 * block per rank); its phases of level 1 are the batches (x = batch number), each
 * with an empty KEEP list and a DELIVER list of P rows, one per receiving rank,
 * holding the batch's steps in ascending ii.
 */
int tuna_plan_create_staggered(tuna_plan_t **out, int P, int radix, int block_count, int l, int g,
                               int elem_size, unsigned flags, const int64_t *sendcounts,
                               const int64_t *sdispls, const int64_t *rdispls,
                               const int64_t *sendbase, const int64_t *recvbase, void *stream);

/*
 * tuna_plan_update_counts - same plan shape, new counts (e.g. routing that changes
 * every step): re-runs the metadata exchange and the prefix sums on the device.
 * Arguments as in tuna_plan_create.  Synchronises `stream` once (for the list
 * totals); when the call returns, the sizes the plan reports are final, while its
 * last kernels (the work partition) may still be running on `stream`: exchange
 * calls order themselves behind them, on whatever stream they are given.  The
 * required workspace size may change; query it again.  The tables are rewritten in place,
 * so the update first waits (on the host) for the exchanges this plan has
 * enqueued, whatever their stream; replays of an exchange captured into a CUDA
 * graph are not tracked and must have finished before the call.  To overlap the
 * re-plan of one batch with the exchange of the previous one, alternate between
 * two plans.
 */
int tuna_plan_update_counts(tuna_plan_t *plan, const int64_t *sendcounts, const int64_t *sdispls,
                            const int64_t *rdispls, const int64_t *sendbase,
                            const int64_t *recvbase, void *stream);

/*
 * tuna_plan_update_counts_device - as tuna_plan_update_counts, for counts that are
 * already in device memory (routing decided on the GPU): the count-metadata
 * exchange and the prefix sums of Sec. III-B/C then start from the device array
 * and nothing crosses the host link but a few totals.
 *   d_sendcounts  DEVICE pointer, P * P int64, [src][dst], in elements; read on
 *                 `stream`; the plan keeps its own copy, so the array may be
 *                 reused as soon as the call returns.
 * The layout is the packed one (what tuna_plan_update_counts does with NULL
 * displacements and bases): every rank's blocks back to back in ascending peer
 * order, the ranks' regions back to back in both buffers.  Region bases, buffer
 * extents and the payload size are computed on the device.
 * Synchronises `stream` once.  The required workspace size may change; query it
 * again.  Waits for this plan's exchanges in flight like tuna_plan_update_counts.
 * Errors: a negative count gives TUNA_ERR_INVALID_ARG; unlike the
 * host-array form, a failed update leaves the plan unusable (its tables have been
 * rewritten; exchange calls return TUNA_ERR_INTERNAL) until an update succeeds.
 * Count or displacement arrays passed to a later exchange call are still
 * compared with the plan's: the first such call copies the counts to the host
 * (one synchronous device-to-host copy).
 */
int tuna_plan_update_counts_device(tuna_plan_t *plan, const int64_t *d_sendcounts, void *stream);

/* Frees the plan's device tables and the plan.  NULL is accepted. */
int tuna_plan_destroy(tuna_plan_t *plan);

/*
 * Workspace (the paper's temporary buffer T, Sec. III-C, sized exactly).
 * tuna_plan_workspace_bytes: bytes needed by tuna_alltoallv on device buffers.
 * tuna_plan_host_staging_bytes: extra bytes needed by tuna_alltoallv_host for
 * device copies of the send and receive buffers.
 * tuna_plan_set_workspace: device pointer, 256-byte aligned, caller-owned, must
 * stay valid while the plan uses it; `bytes` is checked by each exchange call.
 */
int tuna_plan_workspace_bytes(const tuna_plan_t *plan, size_t *bytes);
int tuna_plan_host_staging_bytes(const tuna_plan_t *plan, size_t *bytes);
int tuna_plan_set_workspace(tuna_plan_t *plan, void *dev_ptr, size_t bytes);

/* Extents the plan's layout implies, in bytes: the send buffer is read inside
 * [0, send_bytes), the receive buffer written inside [0, recv_bytes). */
int tuna_plan_extents(const tuna_plan_t *plan, size_t *send_bytes, size_t *recv_bytes,
                      size_t *payload_bytes);

/*
 * tuna_alltoallv - run the plan's TuNA schedule (Algorithm 1, or Sec. IV /
 * Algorithm 3 when g > 1): one fused pack-move-unpack launch per digit phase (all
 * rounds z of one digit position x touch disjoint blocks, so they share it; the
 * self blocks ride along in the first one), and in TUNA_FLAG_CLASSIC_ROTATE mode
 * one rotation launch at the end.
 *
 *   sendbuf, recvbuf   device; must not overlap.
 *   sendcounts, sdispls, recvcounts, rdispls
 *                      host, P*P each, or NULL.  Non-NULL arrays are only checked
 *                      against the plan (TUNA_ERR_COUNT_MISMATCH); the plan's own
 *                      copies drive the kernels.  recvcounts[d*P+s] must equal
 *                      sendcounts[s*P+d].
 * Asynchronous on `stream`; re-runnable; two calls on one plan must not overlap
 * in time (they share the workspace).  With timing off the call only enqueues
 * kernels (no allocation, no synchronisation), so it may be captured into a CUDA
 * graph and replayed while plan, workspace and buffers stay as they were.
 */
int tuna_alltoallv(tuna_plan_t *plan, const void *sendbuf, const int64_t *sendcounts,
                   const int64_t *sdispls, void *recvbuf, const int64_t *recvcounts,
                   const int64_t *rdispls, void *stream);

/*
 * tuna_direct_alltoallv - the linear spread-out exchange (Sec. II-d; the r = P end
 * of Sec. III-C) as ONE launch: every (src, dst) block is read once and written
 * once.  Needs no workspace.  Arguments as tuna_alltoallv.
 */
int tuna_direct_alltoallv(tuna_plan_t *plan, const void *sendbuf, const int64_t *sendcounts,
                          const int64_t *sdispls, void *recvbuf, const int64_t *recvcounts,
                          const int64_t *rdispls, void *stream);

/*
 * tuna_direct_alltoallv_static - the direct exchange for callers that must not
 * allocate device memory.  (The paper has no counterpart: this entry point exists
 * for the library's users, not for the algorithm.)
 *
 * Who needs it: a process whose framework has already claimed the whole GPU for
 * its own memory pool, so that a cudaMalloc from a library fails or fragments the
 * pool; a serving or real-time loop in which cudaMalloc/cudaFree are banned after
 * start-up because they synchronise the device and stall every stream; code that
 * runs under a fixed memory budget and is audited for allocations.  Such callers
 * cannot create a plan (a plan owns descriptor tables obtained with cudaMalloc).
 *
 * This call takes the layout and the buffers in one go and keeps every table it
 * needs (counts, displacements, descriptors, prefix sums, chunk table: about
 * 1.1 MiB) in a fixed array that is part of the library image on every GPU that
 * loads it.  It calls no cudaMalloc, cudaFree or other allocating routine.
 *
 *   P            1 <= P <= TUNA_STATIC_MAX_P, else TUNA_ERR_RANGE.
 *   elem_size, sendcounts, sdispls, rdispls, sendbase, recvbase
 *                host arrays as for tuna_plan_create (NULL = packed).
 *   sendbuf, recvbuf   device; must not overlap.
 *   limit        the work stream (every non-empty block rounded up to 16 bytes plus
 *                16) may not exceed TUNA_STATIC_MAX_CHUNKS * 256 KiB = 4 GiB, else
 *                TUNA_ERR_RANGE; nothing is launched in that case.
 * Errors: besides the limits above, an entry (count, displacement or base) above
 * 2^47 bytes gives TUNA_ERR_RANGE; every size check comes before the buffers are
 * looked at and before anything is enqueued.  The call hands the host arrays to
 * asynchronous copies, which only an eager call may do: on a stream that is being
 * captured it returns TUNA_ERR_INVALID_ARG and records nothing.
 * The first call on a device looks up the array's device address; make that call
 * before starting a stream capture on that device.  All calls share the one array
 * and it keeps the previous call's tables; every table a call reads it first
 * rewrites, so nothing needs clearing, but two calls whose kernels can overlap on
 * the GPU (different streams, no ordering between them) race on it: order them.
 * Asynchronous on `stream`.  Results are byte-identical to tuna_direct_alltoallv.
 */
#define TUNA_STATIC_MAX_P 128
#define TUNA_STATIC_MAX_CHUNKS 16384
int tuna_direct_alltoallv_static(int P, int elem_size, const int64_t *sendcounts,
                                 const int64_t *sdispls, const int64_t *rdispls,
                                 const int64_t *sendbase, const int64_t *recvbase,
                                 const void *sendbuf, void *recvbuf, void *stream);

/*
 * Sharded plans: the ranks spread over several GPUs of one node, one process per GPU.
 *
 * Defines: Sec. IV of the paper with one group per GPU.  The paper's hierarchy exists
 * because links inside a node are faster than links between nodes; here the "node" is
 * one GPU's memory and the slower link is NVLink between GPUs.  Group n (ranks n*l ..
 * n*l + l - 1, l = P / n_gpus) lives on GPU n: its send regions in that GPU's send buffer,
 * its receive regions in that GPU's receive buffer.  The local phases (Sec. IV-A,
 * radix `radix` on the local offset, for all destination groups at once) run inside each
 * GPU; the inter-group phase is the coalesced exchange of Sec. IV-B / Algorithm 3 (one
 * hop, n_gpus - 1 rounds of one super-block of l blocks each) executed as a push: the
 * sending GPU stores every block straight into its place in the receiving GPU's receive
 * buffer.  An inter-group radix below n_gpus would forward super-blocks through third
 * GPUs' memory for no gain (every GPU pair is one hop apart) and is not offered.
 *
 * tuna_shard_plan_create - the plan of GPU `my_gpu`.  Every GPU calls it with the SAME
 * P x P count matrix (all-gather the rows first) and the same displacement arrays.
 *   sendbase[p], recvbase[p]   element offset of rank p's region inside the buffer of
 *                 THE GPU THAT HOLDS RANK p; NULL = that GPU's l regions packed in rank
 *                 order from offset 0.  sdispls / rdispls as in tuna_plan_create.
 *   flags         TUNA_FLAG_CLASSIC_ROTATE and TUNA_FLAG_BULK_COPY are refused
 *                 (TUNA_ERR_INVALID_ARG); TUNA_FLAG_NO_DIRECT is implied.
 *   errors        P not a multiple of n_gpus: TUNA_ERR_BAD_HIERARCHY; n_gpus above 111 or
 *                 my_gpu outside [0, n_gpus): TUNA_ERR_INVALID_ARG; otherwise as
 *                 tuna_plan_create.
 * The plan holds the tables of all P ranks (the metadata work is replicated on every
 * GPU, the data movement is not): its descriptor lists carry a length only where this
 * GPU moves the block.  Introspection reports this GPU's share: a round's `bytes` are the
 * bytes this GPU moves in it, so the sum over the n_gpus plans is the round's volume.
 * tuna_plan_workspace_bytes / tuna_plan_set_workspace: this GPU's workspace (local
 * phases only; the inter-group phase needs none).  tuna_plan_update_counts and
 * tuna_plan_update_counts_device work (the whole P x P matrix, all-gathered; packed
 * bases per GPU; the buffer sizes may change: query tuna_shard_extents again);
 * tuna_alltoallv, tuna_direct_alltoallv, tuna_alltoallv_host and the row exchange
 * return TUNA_ERR_INVALID_ARG for a sharded plan.
 *
 * tuna_shard_extents - bytes of GPU `gpu`'s send and receive buffer that the layout covers.
 *
 * tuna_shard_alltoallv - run this GPU's share.
 *   sendbuf     device, this GPU's send buffer.
 *   recvbufs    HOST array of n_gpus DEVICE pointers: the receive buffer of every GPU as
 *               this process can address it (its own, and the others' mapped through peer
 *               access or an inter-process memory handle).  The caller owns the mappings.
 *   phases      TUNA_SHARD_LOCAL, TUNA_SHARD_GLOBAL or both: the local phases (with the
 *               self blocks) and the inter-group push.  Both in one call is the normal
 *               use; separately they let a caller overlap or inspect the two parts.  The
 *               push reads what the local phases left in the workspace: same stream, or
 *               ordered by the caller.
 * Asynchronous on `stream`; enqueues kernels and, when the addresses in `recvbufs` differ
 * from the previous call's, one small copy of them from a host array the plan keeps (so
 * a call whose addresses changed is not for stream capture).  No kernel waits for another
 * GPU, so the call cannot deadlock whatever the other GPUs do.  It does NOT tell when the other
 * GPUs' stores into this GPU's receive buffer have landed: the caller closes the exchange
 * with a barrier across the GPUs that is ordered behind this call on every GPU's stream
 * (e.g. an NCCL all-reduce on the same stream), and must not reuse a receive buffer
 * before every GPU has passed the previous exchange's barrier.
 *
 * Host-only helpers (no GPU is touched, so they can run before any buffer exists):
 * tuna_shard_layout - the layout rule above, worked out for all GPUs: region bases of
 *   every rank inside its GPU's buffers (sendbase_out, recvbase_out: P values, elements)
 *   and every GPU's buffer sizes (send_bytes, recv_bytes: n_gpus values, bytes); any
 *   output may be NULL.  Use it to size and allocate the buffers whose addresses the
 *   GPUs then exchange.
 * tuna_shard_round_table - the rounds of the sharded schedule in execution order with
 *   what GPU my_gpu sends in each: `level`, `x`, `z` as tuna_plan_round_info; `units` =
 *   blocks (level 0) or super-blocks (level 1) its ranks send, `bytes` their volume.  Up
 *   to `cap` rows are written, *rounds receives the number of rounds.  Level-1 bytes are
 *   this GPU's traffic onto the inter-GPU links.
 * tuna_shard_enable_peer_access - lets kernels of the current device store into
 *   peer_device's memory (cudaDeviceEnablePeerAccess; already enabled counts as success;
 *   TUNA_ERR_INVALID_ARG if the two GPUs have no peer path).
 */
#define TUNA_SHARD_LOCAL 1
#define TUNA_SHARD_GLOBAL 2
int tuna_shard_layout(int P, int n_gpus, int elem_size, const int64_t *sendcounts, const int64_t *sdispls,
                      const int64_t *rdispls, const int64_t *sendbase, const int64_t *recvbase,
                      int64_t *sendbase_out, int64_t *recvbase_out, int64_t *send_bytes,
                      int64_t *recv_bytes);
int tuna_shard_round_table(int P, int n_gpus, int my_gpu, int radix, int elem_size,
                           const int64_t *sendcounts, int cap, int *level, int *x, int *z,
                           int64_t *units, int64_t *bytes, int *rounds);
int tuna_shard_enable_peer_access(int peer_device);
int tuna_shard_plan_create(tuna_plan_t **out, int P, int radix, int n_gpus, int my_gpu, int elem_size,
                           unsigned flags, const int64_t *sendcounts, const int64_t *sdispls,
                           const int64_t *rdispls, const int64_t *sendbase, const int64_t *recvbase,
                           void *stream);
int tuna_shard_extents(const tuna_plan_t *plan, int gpu, size_t *send_bytes, size_t *recv_bytes);
int tuna_shard_alltoallv(tuna_plan_t *plan, const void *sendbuf, void *const *recvbufs, int phases,
                         void *stream);

/*
 * tuna_alltoallv_host - the same exchange on HOST buffers, all on `stream`,
 * returning without synchronising.  `schedule` is TUNA_SCHEDULE_TUNA or
 * TUNA_SCHEDULE_DIRECT, optionally OR-ed with TUNA_HOST_STAGED.
 *   - Both buffers pinned and mapped into the device's address space (cudaHostAlloc
 *     or cudaHostRegister memory under unified addressing), and blocks of 2 KiB or
 *     more on average (or no room for staging in the workspace): the kernels read
 *     host_send and write host_recv in place over the host link, both directions
 *     at once; blocks hop through the device workspace in between.  Needs only
 *     workspace_bytes of workspace; receive-buffer bytes that no block covers are
 *     left untouched.
 *   - Otherwise, or with TUNA_HOST_STAGED: [0, send_bytes) of host_send is copied
 *     to the device, the schedule runs there, and [0, recv_bytes) is copied back
 *     into host_recv.  The workspace must then hold workspace_bytes +
 *     host_staging_bytes, and receive-buffer bytes that no block covers are
 *     overwritten with unspecified values by the copy back.
 */
#define TUNA_HOST_STAGED 0x100
int tuna_alltoallv_host(tuna_plan_t *plan, const void *host_send, void *host_recv, int schedule,
                        void *stream);

/*
 * tuna_plan_set_row_maps, tuna_rows_alltoallv - the exchange of whole rows with a
 * gather in front of it and a scatter behind it, in one pass.
 *
 * The paper has no counterpart: it exchanges contiguous blocks.  A token dispatch
 * (mixture-of-experts routing) holds its rows in token order and wants them in the
 * receiving expert's order; done as gather, exchange, scatter that is three passes
 * over the payload, fused it is one.  The plan's counts and displacements are in
 * rows (elem_size = bytes per row) and describe two VIRTUAL packed buffers; the maps
 * tie them to the caller's real ones.  For every s, d and k < sendcounts[s][d]:
 *   rows_out[scatter_rows[recvbase[d] + rdispls[d][s] + k]]
 *       = rows_in[gather_rows[sendbase[s] + sdispls[s][d] + k]].
 *
 *   gather_rows   DEVICE, one int64 per row of the send layout (send extent in rows),
 *                 or NULL for the identity.  Rows may repeat.
 *   scatter_rows  DEVICE, one int64 per row of the receive layout, or NULL.  Must not
 *                 send two received rows to the same place (not checked; the result
 *                 for such a row is then one of the candidates).
 *   in_rows, out_rows   rows of the two buffers; a map entry outside them, for a row
 *                 that is exchanged, gives TUNA_ERR_RANGE and nothing is moved.
 * set_row_maps reads the maps on `stream` and synchronises it once; the maps may be
 * freed afterwards.  It must be called again after tuna_plan_update_counts.  The
 * row list costs 32 bytes of device memory per exchanged row, owned by the plan.
 * tuna_rows_alltoallv: rows_in, rows_out DEVICE, in_rows / out_rows rows of
 * elem_size bytes, must not overlap (TUNA_ERR_OVERLAP); one launch, asynchronous on
 * `stream`; TUNA_ERR_COUNT_MISMATCH if no maps are set for the current counts.  Rows
 * of rows_out that no block reaches are left untouched.
 */
int tuna_plan_set_row_maps(tuna_plan_t *plan, const int64_t *gather_rows,
                           const int64_t *scatter_rows, int64_t in_rows, int64_t out_rows,
                           void *stream);
int tuna_rows_alltoallv(tuna_plan_t *plan, const void *rows_in, void *rows_out, void *stream);

/*
 * Schedule introspection (host values, filled at plan time).
 * Rounds are the paper's (x, z) pairs in execution order (Sec. III-A); `level` is 0
 * for flat/local rounds and 1 for global rounds; `units` counts blocks sent by all
 * ranks (level 0) or super-blocks of l blocks (level 1); `bytes` is the round's
 * message volume summed over ranks.  Phases are the digit positions.  Every phase
 * has two descriptor lists, selected by `part`: TUNA_PART_KEEP, the blocks that
 * travel on in a later phase and land in the workspace, and TUNA_PART_DELIVER, the
 * blocks that have arrived and land in the receive buffer (empty in
 * TUNA_FLAG_CLASSIC_ROTATE mode); the two lists of a phase share one kernel launch.
 * phase -1 selects the rotation list and -2 the direct list (`part` ignored).
 * A flat plan whose radix is at least P (one digit phase that delivers every
 * block) keeps no separate direct list: tuna_direct_alltoallv then runs that
 * phase's DELIVER list and the self blocks, and phase -2 reports no entries.
 * Plans created with TUNA_FLAG_NO_DIRECT report none either.
 * `entries` descriptor rows, `bytes` moved, `stream_bytes` the padded length of the
 * list's stream (for a KEEP list: the size of its workspace region).
 */
#define TUNA_PART_KEEP 0
#define TUNA_PART_DELIVER 1
int tuna_plan_num_rounds(const tuna_plan_t *plan, int *K);
int tuna_plan_round_info(const tuna_plan_t *plan, int k, int *level, int *x, int *z,
                         int64_t *units, int64_t *bytes);
int tuna_plan_num_phases(const tuna_plan_t *plan, int *n);
int tuna_plan_phase_info(const tuna_plan_t *plan, int phase, int part, int *level, int *x,
                         int64_t *entries, int64_t *bytes, int64_t *stream_bytes);

/*
 * tuna_plan_phase_tables - copy one descriptor list to the host (debug / test hook;
 * synchronises the device).  Each output (host, `cap` rows, may be NULL) receives,
 * per descriptor in receive-side order (rank, then slot): the block length in
 * bytes; its position in the list's stream (the segmented exclusive prefix sum
 * that also partitions the work: lengths rounded up to 16 bytes, plus 16 spare
 * bytes per non-empty block in DELIVER, rotation and direct lists); source and
 * destination as (buffer id << 56 | byte offset), buffer ids 0 = send,
 * 1 = receive, 2 = workspace.  *rows receives the number of descriptors.
 */
int tuna_plan_phase_tables(const tuna_plan_t *plan, int phase, int part, int64_t cap, int64_t *len,
                           int64_t *pos, int64_t *src, int64_t *dst, int64_t *rows);

/* Kernels launched by the last exchange call on this plan (host counter); how many
 * of them ran the small-block build of the mover (kernel names ending in
 * _small_kernel: the build for lists of tiny, mostly skewed or cache-resident
 * blocks) rather than the large-block build; and the kernels launched by every call
 * on this plan since its creation, plan kernels included. */
int tuna_plan_last_launches(const tuna_plan_t *plan, int *launches);
int tuna_plan_last_small_launches(const tuna_plan_t *plan, int *launches);
int tuna_plan_launch_count(const tuna_plan_t *plan, int64_t *launches);

/*
 * Per-kernel timing with the paper's cost components (Sec. V-B lists prepare,
 * metadata, data, replace, rearrange and inter-node cost).  With timing enabled
 * every launch is bracketed by CUDA events on the caller's stream:
 *   TUNA_TIMER_PLAN          metadata exchange + prefix sums (prepare + metadata)
 *   TUNA_TIMER_ROUND_LOCAL   flat / local digit phases (data; "replace" is fused away;
 *                            the first phase's launch also copies the self blocks)
 *   TUNA_TIMER_ROUND_GLOBAL  global digit phases (inter-group cost)
 *   TUNA_TIMER_ROTATE        final rotation when it has a launch of its own (rearrange)
 *   TUNA_TIMER_DIRECT        the single-pass direct exchange
 * tuna_plan_get_timing waits for the recorded events and returns, per kind
 * (arrays of TUNA_TIMER_KINDS, any may be NULL), accumulated milliseconds,
 * launches and payload bytes moved; `reset` non-zero clears the accumulators.
 */
#define TUNA_TIMER_PLAN 0
#define TUNA_TIMER_ROUND_LOCAL 1
#define TUNA_TIMER_ROUND_GLOBAL 2
#define TUNA_TIMER_ROTATE 3
#define TUNA_TIMER_DIRECT 4
#define TUNA_TIMER_KINDS 5
int tuna_plan_enable_timing(tuna_plan_t *plan, int on);
int tuna_plan_get_timing(tuna_plan_t *plan, int reset, double *ms, int64_t *launches,
                         int64_t *bytes);

/* The cudaError_t of the most recent failing runtime call (0 if none). */
int tuna_plan_cuda_error(const tuna_plan_t *plan);

/* Synchronises the device and reports in *gave_up whether any kernel of this plan
 * abandoned a bounded wait (only the TUNA_FLAG_BULK_COPY route waits: on the
 * barriers of its bulk copies); the receive buffer is then incomplete. */
int tuna_plan_device_status(tuna_plan_t *plan, int *gave_up);

/* Static string for a status code. */
const char *tuna_strerror(int status);

/* Library version, major*100 + minor. */
int tuna_version(void);

#ifdef __cplusplus
}
#endif
#endif /* TUNA_H */
