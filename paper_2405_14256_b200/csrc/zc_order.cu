// Ordering of decode calls on a stream: the host-side rules (see zc_order.h).
#include "zc_order.h"

#include "zipcache.h"

#include <algorithm>
#include <cstdint>

namespace {

bool meet(const ZcRange& a, const ZcRange& b) { return a.lo && b.lo && a.lo < b.hi && b.lo < a.hi; }

}  // namespace

ZcOrderSlot zc_order_next(ZcOrderTable* t, ZcFence* fence, const ZcOrderCall& call) {
  ZcOrderSlot s{};
  ZcStreamRec* r = nullptr;
  ZcStreamRec* victim = nullptr;   // an unused record, else the one touched longest ago
  for (int i = 0; i < kZcStreamRecs; ++i) {
    ZcStreamRec* x = &t->rec[i];
    if (x->used && x->st == call.st && x->dev == call.dev) r = x;
    if (!victim || (victim->used && (!x->used || x->age < victim->age))) victim = x;
  }
  bool fresh = false;
  if (!r) {
    r = victim;
    if (r->used) s.drain = r->st;   // its order word changes hands
    r->used = true;
    r->st = call.st;
    r->dev = call.dev;
    r->e = 0;
    fresh = true;
  }
  // a new epoch: this launch is made without early start and so finds the stream drained
  if (fresh || r->e == 0 || r->e >= kZcMaxEpochCalls || r->ws != call.ws || r->ws_bytes != call.ws_bytes ||
      call.need > r->slot_bytes || r->capturing != call.capturing || r->capture_id != call.capture_id) {
    r->tag = (r->tag + 1) & 0xFFFu;
    r->e = 0;
    r->ws = call.ws;
    r->ws_bytes = call.ws_bytes;
    r->K = (int)std::min<size_t>((size_t)ZC_EPOCH_CALLS, call.ws_bytes / call.need);
    r->slot_bytes = (call.ws_bytes / (size_t)r->K) & ~(size_t)255;
    if (r->slot_bytes < call.need) {   // alignment took the room: fewer, larger regions
      r->K = std::max(1, r->K - 1);
      r->slot_bytes = r->K == 1 ? call.ws_bytes : (call.ws_bytes / (size_t)r->K) & ~(size_t)255;
    }
    r->capturing = call.capturing;
    r->capture_id = call.capture_id;
  }
  const int e = r->e;
  const int rec = (int)(r - t->rec);
  s.rec = rec;
  s.tag = r->tag;
  s.e = e;
  s.epoch_start = e == 0;
  s.need_end = e - r->K + 1;
  s.need_start = e - ZC_EPOCH_CALLS + 1;
  for (int i = std::max(0, e - ZC_EPOCH_CALLS + 1); i < e; ++i) {
    const ZcCallRec& o = r->ring[i % ZC_EPOCH_CALLS];
    for (int k = 0; k < 3; ++k) {
      if (meet(call.me.in[k], o.out)) s.need_start = std::max(s.need_start, i + 1);
      if (meet(call.me.out, o.in[k])) s.need_end = std::max(s.need_end, i + 1);
    }
    if (meet(call.me.out, o.out) || (call.collect && o.collected == call.cache))
      s.need_end = std::max(s.need_end, i + 1);
  }
  // an earlier call stored a tail row of this cache or re-compressed its window
  if (e > 0 && fence->rec == rec && fence->tag == r->tag && fence->capturing == call.capturing)
    s.need_start = std::max(s.need_start, fence->e);
  s.slot = e % r->K;
  s.ws_off = (size_t)s.slot * r->slot_bytes;
  if (call.changes_cache) {
    // what this call stores in the cache, the cache's next call reads
    fence->rec = rec;
    fence->tag = r->tag;
    fence->e = e + 1;
    fence->capturing = call.capturing;
  }
  r->ring[e % ZC_EPOCH_CALLS] = call.me;
  r->ring[e % ZC_EPOCH_CALLS].collected = call.collect ? call.cache : nullptr;
  r->e = e + 1;
  r->age = ++t->clock;
  return s;
}

// ---- the model behind zc_order_model_*: the same rules on a table of its own ----
namespace {

constexpr int kModelCaches = 16;
ZcOrderTable g_model;
ZcFence g_model_fence[kModelCaches];
bool g_model_ready = false;

void model_init() {
  if (g_model_ready) return;
  g_model = ZcOrderTable{};
  for (int i = 0; i < kModelCaches; ++i) g_model_fence[i] = ZcFence{-1, 0u, 0, 0};
  g_model_ready = true;
}

}  // namespace

extern "C" void zc_order_model_reset(void) {
  g_model_ready = false;
  model_init();
}

extern "C" int zc_order_model_call(uint64_t stream_id, int cache_id, const uint64_t addr[4],
                                   uint64_t io_bytes, uint64_t kv_bytes, int collect, uint64_t ws_addr,
                                   uint64_t ws_bytes, uint64_t need, uint64_t capture_id, int result[8]) {
  if (!addr || !result || cache_id < 0 || cache_id >= kModelCaches || need == 0 || need > ws_bytes)
    return ZC_EINVAL;
  model_init();
  ZcOrderCall call{};
  call.st = (const void*)(uintptr_t)stream_id;
  call.dev = 0;
  call.me.in[0] = zc_range((const void*)(uintptr_t)addr[0], (size_t)io_bytes);
  call.me.in[1] = zc_range((const void*)(uintptr_t)addr[1], (size_t)kv_bytes);
  call.me.in[2] = zc_range((const void*)(uintptr_t)addr[2], (size_t)kv_bytes);
  call.me.out = zc_range((const void*)(uintptr_t)addr[3], (size_t)io_bytes);
  call.cache = &g_model_fence[cache_id];
  call.collect = collect;
  call.changes_cache = addr[1] != 0;
  call.ws = (const char*)(uintptr_t)ws_addr;
  call.ws_bytes = (size_t)ws_bytes;
  call.need = (size_t)need;
  call.capturing = capture_id != 0;
  call.capture_id = capture_id;
  const ZcOrderSlot s = zc_order_next(&g_model, &g_model_fence[cache_id], call);
  result[0] = s.epoch_start;
  result[1] = s.e;
  result[2] = s.need_start;
  result[3] = s.need_end;
  result[4] = s.slot;
  result[5] = (int)s.tag;
  result[6] = s.rec;
  result[7] = s.drain ? 1 : 0;
  return ZC_OK;
}
