// Internal declarations shared by the plan builder and the mover kernels.
#ifndef TUNA_INTERNAL_H
#define TUNA_INTERNAL_H

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "tuna.h"

// A location is (buffer id << 56) | byte offset inside that buffer.
#define TUNA_BUF_SEND 0
#define TUNA_BUF_RECV 1
#define TUNA_BUF_WORK 2
// Sharded plans (ranks spread over several GPUs): the receive buffer of GPU n.
#define TUNA_BUF_PEER0 16
#define TUNA_MAX_SHARDS (127 - TUNA_BUF_PEER0)  // (a buffer id sits in the top byte of a location and stays positive)
#define TUNA_LOC(buf, off) ((((int64_t)(buf)) << 56) | (int64_t)(off))
#define TUNA_LOC_BUF(loc) ((int)((loc) >> 56))
#define TUNA_LOC_OFF(loc) ((loc) & ((((int64_t)1) << 56) - 1))

#define TUNA_ALIGN 16  // every block in the workspace starts on this boundary
#define TUNA_MOVE_THREADS 256
#define TUNA_MAX_CHUNK_BYTES (256 * 1024)  // stream bytes one CTA handles, at most

// Ranks and slots: rank p = n*Q + q; slot sigma = io*Q + jo names the block whose
// destination is (n + io mod N, q + jo mod Q).  Flat TuNA is N = 1.
struct TunaTopo {
  int P, Q, N;
  int elem;
  // Sharded plan: group n lives on GPU n, and this plan describes the work of GPU
  // shard_me only (shard_n == N GPUs).  Every GPU builds the tables of all P ranks, so
  // that sizes and locations flow through the phases as in a plan for one GPU, but a
  // descriptor is given its length only where this GPU executes it: in a local phase the
  // blocks its own ranks receive, in the global phase the blocks its own ranks send
  // (they are stored straight into the receiving GPU's buffer).  shard_n == 0: one GPU.
  int shard_n, shard_me;
};

// One digit phase: all rounds (x, z), z = 1..radix-1, of one digit position.
struct TunaPhase {
  int level;       // 0: digit of jo (flat / local), 1: digit of io (global)
  int x;           // digit position
  int radix;
  int count;       // Q or N: number of offsets at this level
  int64_t stride;  // radix^x
  int64_t moving;  // offsets below count whose digit x is non-zero
  int64_t per_rank;  // blocks a rank receives in this phase
  int64_t finals;    // the first `finals` of them (in slot order) have arrived and are delivered
  int64_t stats_off; // first of `radix` counters in the stats array
  // Staggered inter-group exchange: this "phase" is one batch of steps [stag_lo,
  // stag_hi) of the step index ii = gi*Q + gr; every block it moves has arrived.
  // stag_hi == 0 for an ordinary digit phase.
  int stag_lo, stag_hi;
};

// How a list's stream positions are spaced.
//   KEEP:    pos = exclusive prefix sum of the lengths rounded up to 16.  The stream
//            is the destination itself (a region of the workspace).
//   DELIVER: 16 further bytes per non-empty block, so that a block can sit in a
//            staging buffer at its destination's alignment whatever that is; the
//            stream only partitions the work.
enum TunaListKind { TUNA_LIST_KEEP = 0, TUNA_LIST_DELIVER = 1 };

// A list of copy descriptors in receive-side order with its work partition.
struct TunaList {
  int kind = TUNA_LIST_KEEP;
  int64_t n = 0;          // descriptors
  int64_t *len = nullptr; // bytes
  int64_t *pos = nullptr; // n + 1 stream positions (pos[n] = total)
  int64_t *src = nullptr; // location
  int64_t *dst = nullptr; // location (DELIVER lists only)
  int32_t *chunk_first = nullptr;
  int64_t chunk_cap = 0;  // allocated entries of chunk_first
  int64_t total = 0;      // stream bytes (host copy)
  int64_t bytes = 0;      // bytes moved (host copy)
  int64_t unaligned_bytes = 0;  // ... of which in blocks whose source and destination differ modulo 16
  int64_t chunk = 0;      // bytes of stream per CTA
  int64_t nchunks = 0;
  bool small_blocks = false;  // runs the small-block kernel build (tiny or mostly skewed blocks)
};

// Device view of one list.
struct TunaListArgs {
  const int64_t *len, *pos, *src, *dst;
  const int32_t *chunk_first;
  int64_t n, total, chunk, nchunks;  // nchunks == 0: the list takes no part in the launch
  int skewed;  // most of the list's bytes sit in blocks whose source and destination differ modulo 16
};

// One launch moves up to three independent lists: the CTAs [0, keep.nchunks) take
// the KEEP list, the next del.nchunks the first DELIVER list, the rest the second.
struct TunaMoveArgs {
  TunaListArgs keep;  // blocks of a digit phase that travel on (workspace)
  TunaListArgs del;   // blocks of a digit phase that have arrived, or the direct list
  TunaListArgs rot;   // rotation list (self blocks, or every block in classic mode)
  char *base[3];
  char *const *peer;  // sharded plans: device array of the GPUs' receive buffers (null otherwise)
  int64_t extent[3];  // bytes of each buffer that may be accessed, from its base
  int64_t keep_base;  // workspace offset of stream position 0 of the KEEP list
  int *error;         // device flag raised when a bounded wait inside a kernel gave up (may be null)
  int bulk_off;       // in: non-zero asks for the bulk-copy route; the launcher turns it into the offset
                      // of the staging area in dynamic shared memory (0 = route off)
  int wait_first;     // set by the launcher: wait for the previous kernel of the stream before the first
                      // table read (the first launch of an exchange, which may follow the plan kernels)
};

enum TunaMoveKernel {
  TUNA_K_ROUND = 0,   // a digit phase (with the self blocks riding along in the first one)
  TUNA_K_ROTATE = 1,  // the rotation list alone
  TUNA_K_DIRECT = 2   // single-pass direct exchange
};

// Launches one mover kernel (tuna_move.cu).  `small_blocks` picks the build tuned
// for lists whose blocks are far smaller than a chunk.  Every launch may be scheduled
// while the previous kernel of the stream drains; `early_start` also lets its CTAs
// read the plan's tables before they wait for that kernel: only for a launch that
// cannot follow the kernels that write those tables directly (a later launch of an
// exchange, or the first one when an earlier exchange has already run behind the
// last update); otherwise it waits before its first table read.
cudaError_t tuna_launch_move(int kernel, const TunaMoveArgs &a, bool small_blocks, bool early_start,
                             cudaStream_t stream);

#endif
