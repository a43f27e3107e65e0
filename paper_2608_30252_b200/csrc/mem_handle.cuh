// Host handle of the draft memory and the layout of its device workspace.
#pragma once

#include <vector>

#include "common.cuh"

namespace masw {

constexpr int kMaxSplits = 64;      // upper bound on split-K partials per (sequence, KV head); equals kMaxSplitsDev
constexpr int kCtaBudget = 320;     // CTAs assumed co-resident when sizing split-K scratch
constexpr int kProjKSplit = 16;     // k-splits of the slot projection

struct WsLayout {
  size_t off_t, off_slots, off_status, off_tickets_attn, off_tickets_proj, off_part_o, off_part_ml, off_proj_part, off_part_slot;
  size_t total;
  int splits_max, rows_max;
};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static inline int ring_capacity(const masw_config& c) {
  return static_cast<int>(align_up(static_cast<size_t>(c.window) + c.rollback + c.gamma_max, 64));
}

static inline int entries_per_head(const masw_config& c) { return c.sink + c.max_slots + ring_capacity(c); }

static inline int splits_cap(int batch, int n_kv_heads) {
  int s = (kCtaBudget + batch * n_kv_heads - 1) / (batch * n_kv_heads);
  return s < 1 ? 1 : (s > kMaxSplits ? kMaxSplits : s);
}

static inline WsLayout ws_layout(const masw_config& c) {
  WsLayout L;
  const int G = c.n_q_heads / c.n_kv_heads;
  const int rows = (c.gamma_max + 1) * G;
  L.rows_max = static_cast<int>(align_up(rows, 16));
  L.splits_max = splits_cap(c.batch, c.n_kv_heads);
  size_t off = 0;
  L.off_t = off;            off += align_up(sizeof(int) * c.batch, 256);
  L.off_slots = off;        off += align_up(sizeof(int) * c.batch, 256);
  L.off_status = off;       off += 256;
  L.off_tickets_attn = off; off += align_up(sizeof(int) * (kMaxSplits + 1) * c.batch * c.n_kv_heads, 256);
  L.off_tickets_proj = off; off += align_up(sizeof(int) * 2 * c.n_kv_heads, 256);
  L.off_part_o = off;
  off += align_up(sizeof(unsigned long long) * c.batch * c.n_kv_heads * L.splits_max * L.rows_max * c.head_dim, 256);
  L.off_part_ml = off;
  off += align_up(sizeof(unsigned long long) * c.batch * c.n_kv_heads * L.splits_max * L.rows_max * 2, 256);
  L.off_proj_part = off;
  off += align_up(sizeof(float) * kProjKSplit * c.batch * 2 * c.n_kv_heads * c.head_dim, 256);
  L.off_part_slot = off;
  off += align_up(sizeof(unsigned long long) * c.batch * c.n_kv_heads * L.splits_max * 2 * c.head_dim, 256);
  L.total = off;
  return L;
}

}  // namespace masw

struct masw_mem {
  masw_config cfg;
  int G, ring_cap, n_cap;
  float scale;
  double rope_base;
  uint8_t* arena;
  size_t arena_bytes;
  size_t tensor_elems;  // elements of one K (or V) tensor of one layer: B * Hkv * n_cap * D
  uint8_t* ws;
  masw::WsLayout L;
  int* d_t;
  int* d_slots;
  int* d_status;
  int* d_tickets_attn;
  int* d_tickets_proj;
  unsigned long long* d_part_o;   // tagged 64-bit records (payload, epoch tag)
  unsigned long long* d_part_ml;
  float* d_proj_part;
  unsigned long long* d_part_slot;
  std::vector<CUtensorMap> tmK32, tmV32, tmK64, tmV64;  // per layer, box of 32 / 64 entries
  int slots_upper;  // host-side upper bound on any sequence's committed slot count
  // True while the last call on this handle was a draft attention launch: such a launch waits for its
  // predecessor before it lets its successor start, and writes neither the counters nor another layer's K/V,
  // so the next layer's launch may read those ahead of its own wait.  Every call that writes the counters
  // or the arena through another path (mem_update, mem_load, mem_advance, mem_rollback, mem_set_state, the
  // prefill import) clears it.
  bool kv_clean = false;
  // A counter update that was only noted (mem_advance_deferred): t[b] + pend_t and min(n_slots[b] + pend_m,
  // max_slots) are the counters in force.  Draft attention launches and mem_rollback take the two numbers as
  // launch parameters; every other call that reads or writes the counters applies them first (flush_counters).
  int pend_t = 0, pend_m = 0;

  __nv_bfloat16* k_layer(int layer) const {
    return reinterpret_cast<__nv_bfloat16*>(arena) + static_cast<size_t>(layer) * 2 * tensor_elems;
  }
  __nv_bfloat16* v_layer(int layer) const { return k_layer(layer) + tensor_elems; }
};

namespace masw {
// Applies a deferred counter update with one launch of the advance kernel (no-op when nothing is pending).
int flush_counters(masw_mem* mem, cudaStream_t st);
}  // namespace masw
