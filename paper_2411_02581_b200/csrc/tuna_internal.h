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
#define TUNA_LOC(buf, off) ((((int64_t)(buf)) << 56) | (int64_t)(off))
#define TUNA_LOC_BUF(loc) ((int)((loc) >> 56))
#define TUNA_LOC_OFF(loc) ((loc) & ((((int64_t)1) << 56) - 1))

#define TUNA_ALIGN 16  // every block in the workspace starts on this boundary
#define TUNA_MOVE_THREADS 256

// Ranks and slots: rank p = n*Q + q; slot sigma = io*Q + jo names the block whose
// destination is (n + io mod N, q + jo mod Q).  Flat TuNA is N = 1.
struct TunaTopo {
  int P, Q, N;
  int elem;
};

// One digit phase: all rounds (x, z), z = 1..radix-1, of one digit position.
struct TunaPhase {
  int level;       // 0: digit of jo (flat / local), 1: digit of io (global)
  int x;           // digit position
  int radix;
  int count;       // Q or N: number of offsets at this level
  int64_t stride;  // radix^x
  int64_t moving;  // offsets below count whose digit x is non-zero
  int64_t per_rank;  // descriptors per receiving rank
  int64_t stats_off; // first of `radix` counters in the stats array
};

// A list of copy descriptors in receive-side order with its work partition.
struct TunaList {
  int64_t n = 0;          // descriptors
  int64_t *len = nullptr; // bytes
  int64_t *pos = nullptr; // exclusive prefix sum of 16-byte-padded lengths
  int64_t *src = nullptr; // location
  int64_t *dst = nullptr; // location
  int32_t *chunk_first = nullptr;
  int64_t chunk_cap = 0;  // allocated entries of chunk_first
  int64_t total = 0;      // padded stream bytes (host copy)
  int64_t bytes = 0;      // bytes moved (host copy)
  int64_t chunk = 0;      // bytes of stream per CTA
  int64_t nchunks = 0;
};

struct TunaMoveArgs {
  const int64_t *len, *pos, *src, *dst;
  const int32_t *chunk_first;
  int64_t n, total, chunk, nchunks;
  char *base[3];
  int64_t extent[3];  // bytes of each buffer that may be accessed, from its base
};

enum TunaMoveKind { TUNA_MOVE_ROUND = 0, TUNA_MOVE_ROTATE = 1, TUNA_MOVE_DIRECT = 2 };

// Launches the fused pack-move-unpack kernel over one list (tuna_move.cu).
cudaError_t tuna_launch_move(int kind, const TunaMoveArgs &a, cudaStream_t stream);

#endif
