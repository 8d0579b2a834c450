// Host-side bookkeeping that orders decode calls issued on one stream.  Pure host code: no
// CUDA call is made here, so the rules can be exercised without a device.
//
// Calls launched on a stream since the last launch made without early start form an epoch and
// may be in flight together.  Call e of an epoch uses region e mod K of the workspace and
// arrival counter e mod K.  Its kernel waits until
//   need_start earlier calls of the epoch have completed before it reads its inputs, and
//   need_end   earlier calls have completed before it writes partials, the output and the
//              window statistics.
// The conflicts are found by comparing address ranges with the last ZC_EPOCH_CALLS calls;
// anything older is covered by waiting for call e - ZC_EPOCH_CALLS.
#pragma once

#include <cstddef>

#include "zc_internal.h"

struct ZcRange { const char* lo; const char* hi; };

struct ZcCallRec {
  ZcRange in[3];                    // q, k_new, v_new
  ZcRange out;
  const void* collected;            // cache whose window statistics the call updates
};

struct ZcStreamRec {
  const void* st;                   // the stream (compared only)
  bool used;
  int dev;
  unsigned tag;                     // epoch tag, 12 bits
  int e;                            // calls launched in the current epoch
  int K;                            // workspace regions / arrival counters in use
  const char* ws;
  size_t ws_bytes, slot_bytes;
  int capturing;
  unsigned long long capture_id;
  ZcCallRec ring[ZC_EPOCH_CALLS];
  unsigned long long age;
};

constexpr int kZcStreamRecs = 16;   // one pair of order words per record
constexpr int kZcMaxEpochCalls = (1 << 20) - 1;   // e shares a 32-bit word with the tag

struct ZcOrderTable {
  ZcStreamRec rec[kZcStreamRecs];
  unsigned long long clock;
};

// One decode call as the ordering sees it.
struct ZcOrderCall {
  const void* st;
  int dev;
  ZcCallRec me;
  const void* cache;
  int collect;
  int changes_cache;                // the call stores a tail row or re-compresses the window
  const char* ws;
  size_t ws_bytes;
  size_t need;                      // workspace bytes of this call
  int capturing;
  unsigned long long capture_id;
};

struct ZcOrderSlot {
  int rec;                          // index of the stream record (selects the order word)
  unsigned tag;
  int e, need_start, need_end, epoch_start;
  int slot;                         // workspace region and arrival counter
  size_t ws_off;
  const void* drain;                // non-null: that stream's record changed hands; it must be
                                    // drained before this call is launched
};

static inline ZcRange zc_range(const void* p, size_t n) {
  return ZcRange{(const char*)p, p ? (const char*)p + n : nullptr};
}

// Books the next call of a stream and returns what its kernel has to wait for.
ZcOrderSlot zc_order_next(ZcOrderTable* t, ZcFence* fence, const ZcOrderCall& call);
