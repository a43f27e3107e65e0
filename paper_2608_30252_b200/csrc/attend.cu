// draft_attend and verify_attend: host-side validation, split sizing and launch of the shared
// flash-decode kernel.
#include <mutex>
#include <vector>

#include <type_traits>

#include "attend_draft_kernel.cuh"
#include "attend_kernel.cuh"
#include "attend_tc_kernel.cuh"
#include "mem_handle.cuh"

namespace masw {

#ifdef MASW_TRACE
// developer build only (never part of the product library): a device buffer that receives per-CTA phase
// timestamps, a shortened limit for the kernels' bounded waits, and the index of one tile whose copy is left
// out so that such a wait runs out (the way the give-up path is tested without any fault)
static long long* g_trace = nullptr;
static long long g_trace_stride = 0;   // words by which the record area advances from one launch to the next (0: all launches share it)
static long long g_trace_launch = 0;
static int g_wait_limit = kWaitLimit;
static int g_drop_tile = -1;
static int g_debug_flags = 0;
static void apply_debug(AttendParams& p) {
  p.debug_flags = g_debug_flags;
  if (g_debug_flags & 4) p.early = 0;
  p.trace = g_trace ? g_trace + (g_trace_launch++) * g_trace_stride : nullptr;
  p.wait_limit = g_wait_limit;
  p.drop_tile = g_drop_tile;
}
#else
static void apply_debug(AttendParams&) {}
#endif

// One kernel instance: up to splits_max independent CTAs per (sequence, KV head), CT CTAs per SM.
template <int D, int MT, int EW, int TE, int NSTAGE, int CT>
static int launch_attend(const CUtensorMap& tmK, const CUtensorMap& tmV, AttendParams p, int B, int Hkv,
                         int tiles_upper, int splits_max, cudaStream_t st) {
  using C = AttendCfg<D, MT, EW, TE, NSTAGE>;
  auto kern = attend_kernel<D, MT, EW, TE, NSTAGE, CT>;
  static PerDeviceOnce once;
  { const int rc = set_smem_once(kern, C::kSmemBytes, once); if (rc != MASW_OK) return rc; }
  p.early = 0;
  int splits = (sm_count() * CT) / (B * Hkv);
  if (splits > splits_max) splits = splits_max;
  if (splits > tiles_upper) splits = tiles_upper;
  if (splits < 1) splits = 1;
  p.splits = splits;
  p.wait_limit = kWaitLimit;
  apply_debug(p);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(splits, Hkv, B);
  cfg.blockDim = dim3(C::kThreads, 1, 1);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = st;
  // the splits of one (sequence, KV head) wait for one another: a cooperative launch guarantees that
  // all CTAs are resident together (splits * B * Hkv <= SM count by construction when splits > 1)
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (splits > 1) { attr[na].id = cudaLaunchAttributeCooperative; attr[na].val.cooperative = 1; ++na; }
  // the kernel may be set up while its predecessor in the stream drains: it touches no global memory before
  // its griddepcontrol.wait
  attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization; attr[na].val.programmaticStreamSerializationAllowed = 1; ++na;
  cfg.attrs = attr;
  cfg.numAttrs = na;
  MASW_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmK, tmV, p));
  count_launch();
  return MASW_OK;
}

// The draft's decode launch for up to eight query rows per KV head: one CTA per SM and launch, but a footprint
// that lets the next layer's CTAs become resident beside this layer's (see attend_draft_kernel.cuh).
template <int D, bool PACK, bool SLOT>
static int launch_attend_draft(const CUtensorMap& tmK, const CUtensorMap& tmV, AttendParams p, int B, int Hkv,
                               int tiles_upper, int splits_max, cudaStream_t st) {
  using C = DraftCfg<D>;
  auto kern = attend_draft_kernel<D, PACK, SLOT>;
  static PerDeviceOnce once;
  {
    const int dev = current_device();
    if (!once.done[dev].load(std::memory_order_acquire)) {
      // the whole configurable array as shared memory, so that two 113 KB CTAs fit on an SM
      MASW_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared));
    }
    const int rc = set_smem_once(kern, C::kSmemBytes, once);
    if (rc != MASW_OK) return rc;
  }
  int splits = sm_count() / (B * Hkv);
  if (splits > splits_max) splits = splits_max;
  if (splits > tiles_upper) splits = tiles_upper;
  if (splits < 1) splits = 1;
  p.splits = splits;
  p.wait_limit = kWaitLimit;
  apply_debug(p);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(splits, Hkv, B);
  cfg.blockDim = dim3(C::kThreads, 1, 1);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (splits > 1) { attr[na].id = cudaLaunchAttributeCooperative; attr[na].val.cooperative = 1; ++na; }
  attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization; attr[na].val.programmaticStreamSerializationAllowed = 1; ++na;
  cfg.attrs = attr;
  cfg.numAttrs = na;
  MASW_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmK, tmV, p));
  count_launch();
  return MASW_OK;
}

// tcgen05 / TMEM kernel (head_dim 128): query rows padded to NQ, rings of NK K tiles and NV V tiles (32 KB each)
template <int NQ, int NK, int NV, bool FP8 = false>
static int launch_attend_tc(const CUtensorMap& tmK, const CUtensorMap& tmV, const CUtensorMap& tmKn, const CUtensorMap& tmVn,
                            AttendParams p, int B, int Hkv, int tiles_upper, int splits_max, cudaStream_t st) {
  using C = TcCfg<NQ, NK, NV, FP8>;
  auto kern = attend_tc_kernel<NQ, NK, NV, FP8>;
  static PerDeviceOnce once;
  { const int rc = set_smem_once(kern, C::kSmemBytes, once); if (rc != MASW_OK) return rc; }
  int splits = sm_count() / (B * Hkv);
  if (splits > splits_max) splits = splits_max;
  if (splits > tiles_upper) splits = tiles_upper;
  if (splits < 1) splits = 1;
  p.splits = splits;
  p.wait_limit = kWaitLimit;
  apply_debug(p);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(splits, Hkv, B);
  cfg.blockDim = dim3(C::kThreads, 1, 1);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  int na = 0;
  if (splits > 1) { attr[na].id = cudaLaunchAttributeCooperative; attr[na].val.cooperative = 1; ++na; }
  attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization; attr[na].val.programmaticStreamSerializationAllowed = 1; ++na;
  cfg.attrs = attr;
  cfg.numAttrs = na;
  MASW_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmK, tmV, tmKn, tmVn, p));
  count_launch();
  return MASW_OK;
}

// tile entries used by each (D, MT) instance; must match the dispatch below
static int tile_entries(int D, int mt) {
  if (D == 64) return 64;
  return mt <= 2 ? 32 : 64;
}

static int dispatch_attend(int D, int mt, const CUtensorMap& tmK, const CUtensorMap& tmV, const AttendParams& p,
                           int B, int Hkv, int entries_upper, int nseg_upper, int splits_max, cudaStream_t st) {
  const int te = tile_entries(D, mt);
  const int tiles_upper = (entries_upper + te - 1) / te + nseg_upper;
  // template arguments: D, MT, EW, TE, NSTAGE, CTAs per SM
  if (D == 64) {
    switch (mt) {
      case 1: return launch_attend<64, 1, 4, 64, 12, 1>(tmK, tmV, p, B, Hkv, tiles_upper, splits_max, st);
      case 2: return launch_attend<64, 2, 4, 64, 12, 1>(tmK, tmV, p, B, Hkv, tiles_upper, splits_max, st);
      case 3: return launch_attend<64, 3, 3, 64, 12, 1>(tmK, tmV, p, B, Hkv, tiles_upper, splits_max, st);
      case 4: return launch_attend<64, 4, 2, 64, 12, 1>(tmK, tmV, p, B, Hkv, tiles_upper, splits_max, st);
    }
  } else if (D == 128) {
    switch (mt) {
      case 1: return launch_attend<128, 1, 4, 32, 12, 1>(tmK, tmV, p, B, Hkv, tiles_upper, splits_max, st);
      case 2: return launch_attend<128, 2, 4, 32, 12, 1>(tmK, tmV, p, B, Hkv, tiles_upper, splits_max, st);
      case 3: return launch_attend<128, 3, 3, 64, 6, 1>(tmK, tmV, p, B, Hkv, tiles_upper, splits_max, st);
      case 4: return launch_attend<128, 4, 2, 64, 6, 1>(tmK, tmV, p, B, Hkv, tiles_upper, splits_max, st);
    }
  }
  set_error("unsupported attention shape: head_dim %d, %d row blocks", D, mt);
  return MASW_EINVAL;
}

// ---- verify_attend: scratch layout and tensor-map cache -------------------------------------------
struct VerifyWs {
  size_t off_tickets, off_part_o, off_part_ml, total;
  int splits_max, rows_max;
};

static VerifyWs verify_ws(int B, int Hkv, int G, int D, int T) {
  VerifyWs w;
  w.rows_max = (T * G <= 32) ? 32 : 64;   // the tcgen05 kernel pads the query rows to 32 or 64
  w.splits_max = splits_cap(B, Hkv);
  size_t off = 0;
  w.off_tickets = off; off += align_up(sizeof(int) * (kMaxSplitsDev + 1) * B * Hkv, 256);
  w.off_part_o = off;  off += align_up(sizeof(unsigned long long) * B * Hkv * w.splits_max * w.rows_max * D, 256);
  w.off_part_ml = off; off += align_up(sizeof(unsigned long long) * B * Hkv * w.splits_max * w.rows_max * 2, 256);
  w.total = off;
  return w;
}

struct MapKey {
  const void* k; const void* v;
  int64_t sb, sh, sn;
  int B, Hkv, D, cap, box;
  bool operator==(const MapKey& o) const {
    return k == o.k && v == o.v && sb == o.sb && sh == o.sh && sn == o.sn && B == o.B && Hkv == o.Hkv && D == o.D &&
           cap == o.cap && box == o.box;
  }
};
struct MapEntry { MapKey key; CUtensorMap tk, tv; };
static std::mutex g_map_mu;
static std::vector<MapEntry> g_maps;

int get_kv_maps(const masw_kv_desc& kv, int box, CUtensorMap* tk, CUtensorMap* tv) {
  MapKey key{kv.k, kv.v, kv.stride_b, kv.stride_h, kv.stride_n, kv.batch, kv.n_kv_heads, kv.head_dim, kv.capacity, box};
  std::lock_guard<std::mutex> lock(g_map_mu);
  for (const MapEntry& e : g_maps) {
    if (e.key == key) { *tk = e.tk; *tv = e.tv; return MASW_OK; }
  }
  MapEntry e;
  e.key = key;
  int rc = encode_kv_tensor_map(&e.tk, kv.k, kv.head_dim, kv.capacity, kv.n_kv_heads, kv.batch, kv.stride_n, kv.stride_h,
                                kv.stride_b, box);
  if (rc != MASW_OK) return rc;
  rc = encode_kv_tensor_map(&e.tv, kv.v, kv.head_dim, kv.capacity, kv.n_kv_heads, kv.batch, kv.stride_n, kv.stride_h,
                            kv.stride_b, box);
  if (rc != MASW_OK) return rc;
  if (g_maps.size() >= 256) g_maps.erase(g_maps.begin());
  g_maps.push_back(e);
  *tk = e.tk; *tv = e.tv;
  return MASW_OK;
}

}  // namespace masw

using namespace masw;

#ifdef MASW_TRACE
extern "C" void masw_debug_set_trace(void* device_buffer, long long stride_words) {
  g_trace = static_cast<long long*>(device_buffer);
  g_trace_stride = stride_words;
  g_trace_launch = 0;
}
extern "C" void masw_debug_set_wait(int wait_limit, int drop_tile) {
  g_wait_limit = wait_limit > 0 ? wait_limit : kWaitLimit;
  g_drop_tile = drop_tile;
}
extern "C" void masw_debug_set_flags(int flags) { g_debug_flags = flags; }
#endif

struct SlotInputs {
  const void* h_g = nullptr;
  const void* Wk_g = nullptr;
  const void* Wv_g = nullptr;
  const int32_t* slot_pos = nullptr;
  const uint8_t* active = nullptr;
};

static int draft_attend_impl(masw_mem* mem, int layer, const void* k_raw, const void* v_raw, const SlotInputs& slot,
                             const void* q, int n_q, int last_row_is_slot, float* o, float* lse, void* o_bf16,
                             void* stream, const char* who) {
  MASW_REQUIRE(mem != nullptr && q != nullptr && o != nullptr, MASW_EINVAL, "%s: null argument", who);
  MASW_REQUIRE(layer >= 0 && layer < mem->cfg.n_layers, MASW_EINVAL, "%s: layer %d out of range", who, layer);
  MASW_REQUIRE(last_row_is_slot == 0 || last_row_is_slot == 1, MASW_EINVAL, "%s: last_row_is_slot must be 0/1", who);
  MASW_REQUIRE(n_q >= 1 && n_q - last_row_is_slot <= mem->cfg.gamma_max, MASW_EINVAL,
               "%s: n_q %d outside [1, gamma_max + slot row]", who, n_q);
  MASW_REQUIRE(n_q * mem->G <= 64 && n_q * mem->G <= mem->L.rows_max, MASW_EINVAL,
               "%s: n_q * group size = %d exceeds the query tile", who, n_q * mem->G);
  MASW_REQUIRE(aligned16(q) && aligned16(o) && aligned16(o_bf16) && aligned16(k_raw) && aligned16(v_raw), MASW_EALIGN,
               "%s: pointers must be 16-byte aligned", who);
  const masw_config& c = mem->cfg;
  const int mt = (n_q * mem->G + 15) / 16;
  AttendParams p{};
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k_raw = static_cast<const __nv_bfloat16*>(k_raw);
  p.v_raw = static_cast<const __nv_bfloat16*>(v_raw);
  p.k_base = mem->k_layer(layer); p.v_base = mem->v_layer(layer);
  p.stride_h = static_cast<long long>(mem->n_cap) * c.head_dim;
  p.stride_b = p.stride_h * c.n_kv_heads;
  p.h_g = static_cast<const __nv_bfloat16*>(slot.h_g);
  p.Wk_g = static_cast<const __nv_bfloat16*>(slot.Wk_g);
  p.Wv_g = static_cast<const __nv_bfloat16*>(slot.Wv_g);
  p.slot_pos = slot.slot_pos; p.active = slot.active;
  p.part_slot = mem->d_part_slot; p.d_model = c.d_model; p.rope_base = mem->rope_base;
  p.o = o; p.lse = lse; p.o_bf16 = static_cast<__nv_bfloat16*>(o_bf16);
  p.part_o = mem->d_part_o; p.part_ml = mem->d_part_ml;
  p.tickets = mem->d_tickets_attn; p.status = mem->d_status;
  p.t = mem->d_t; p.n_slots = mem->d_slots; p.kv_len = nullptr;
  p.dt = mem->pend_t; p.dm = mem->pend_m;   // a deferred counter update travels as launch parameters
  p.n_q = n_q; p.last_row_is_slot = last_row_is_slot;
  p.G = mem->G; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads;
  p.S = c.sink; p.W = c.window; p.ring_cap = mem->ring_cap; p.max_slots = c.max_slots;
  p.capacity = mem->n_cap;
  p.scale_log2e = mem->scale * 1.4426950408889634f;
  const int entries_upper = c.sink + std::min(mem->slots_upper + 1, c.max_slots) + c.window + n_q;
  const bool te32 = (tile_entries(c.head_dim, mt) == 32);
  const CUtensorMap& tk = te32 ? mem->tmK32[layer] : mem->tmK64[layer];
  const CUtensorMap& tv = te32 ? mem->tmV32[layer] : mem->tmV64[layer];
  int rc;
  if (n_q * mem->G <= 8) {
    // a slot row whose slot was written by mem_update (not by this launch) reads that entry: never ahead of the wait
    p.early = (mem->kv_clean && !(last_row_is_slot && slot.h_g == nullptr)) ? 1 : 0;
    // a launch that must wait first may still ask its tiles into L2 early, if they will still be there when it runs
    const long long kv_bytes = 4LL * entries_upper * c.batch * c.n_kv_heads * c.head_dim;
    p.guess_hint = (kv_bytes <= (48LL << 20)) ? 1 : 0;
    const int te = (c.head_dim == 64) ? DraftCfg<64>::TE : DraftCfg<128>::TE;   // equals tile_entries(head_dim, 1): same tensor maps
    const int tiles_upper = (entries_upper + te - 1) / te + 4;
    // at most four rows: the instance that packs both bf16 terms of the probabilities into one MMA's columns
    const bool pack = n_q * mem->G <= 4;
    const cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool fused_slot = p.h_g != nullptr;   // the instance with the boundary step's slot materialisation
    auto go = [&](auto d, auto pk, auto sl) {
      return launch_attend_draft<decltype(d)::value, decltype(pk)::value, decltype(sl)::value>(
          tk, tv, p, c.batch, c.n_kv_heads, tiles_upper, mem->L.splits_max, st);
    };
    using std::integral_constant;
    using T = std::true_type;
    using F = std::false_type;
    if (c.head_dim == 64) {
      using Dn = integral_constant<int, 64>;
      rc = pack ? (fused_slot ? go(Dn{}, T{}, T{}) : go(Dn{}, T{}, F{})) : (fused_slot ? go(Dn{}, F{}, T{}) : go(Dn{}, F{}, F{}));
    } else {
      using Dn = integral_constant<int, 128>;
      rc = pack ? (fused_slot ? go(Dn{}, T{}, T{}) : go(Dn{}, T{}, F{})) : (fused_slot ? go(Dn{}, F{}, T{}) : go(Dn{}, F{}, F{}));
    }
  } else {
    rc = dispatch_attend(c.head_dim, mt, tk, tv, p, c.batch, c.n_kv_heads, entries_upper, 4, mem->L.splits_max,
                         static_cast<cudaStream_t>(stream));
  }
  // either kernel waits for its predecessor before it lets a successor start and writes neither the counters
  // nor another layer's K/V: the next layer's launch may read those early
  mem->kv_clean = (rc == MASW_OK);
  return rc;
}

extern "C" int draft_attend(masw_mem* mem, int layer, const void* q, int n_q, int last_row_is_slot, float* o,
                            float* lse, void* o_bf16, void* stream) {
  return draft_attend_impl(mem, layer, nullptr, nullptr, SlotInputs{}, q, n_q, last_row_is_slot, o, lse, o_bf16, stream,
                           "draft_attend");
}

extern "C" int draft_append_attend(masw_mem* mem, int layer, const void* k_raw, const void* v_raw, const void* q,
                                   int n_q, int last_row_is_slot, float* o, float* lse, void* o_bf16, void* stream) {
  MASW_REQUIRE(k_raw != nullptr && v_raw != nullptr, MASW_EINVAL, "draft_append_attend: k_raw and v_raw must be given");
  MASW_REQUIRE(n_q - (last_row_is_slot ? 1 : 0) >= 1, MASW_EINVAL, "draft_append_attend: needs at least one raw row");
  return draft_attend_impl(mem, layer, k_raw, v_raw, SlotInputs{}, q, n_q, last_row_is_slot, o, lse, o_bf16, stream,
                           "draft_append_attend");
}

extern "C" int draft_boundary_attend(masw_mem* mem, int layer, const void* k_raw, const void* v_raw, const void* h_g,
                                     const void* Wk_g, const void* Wv_g, const int32_t* slot_pos, const uint8_t* active,
                                     const void* q, int n_q, float* o, float* lse, void* o_bf16, void* stream) {
  MASW_REQUIRE(mem != nullptr, MASW_EINVAL, "draft_boundary_attend: null handle");
  MASW_REQUIRE(k_raw != nullptr && v_raw != nullptr && h_g != nullptr && Wk_g != nullptr && Wv_g != nullptr &&
                   slot_pos != nullptr,
               MASW_EINVAL, "draft_boundary_attend: k_raw, v_raw, h_g, Wk_g, Wv_g and slot_pos must all be given");
  MASW_REQUIRE(n_q >= 2, MASW_EINVAL, "draft_boundary_attend: needs at least one raw row and the slot row");
  MASW_REQUIRE(aligned16(h_g) && aligned16(Wk_g) && aligned16(Wv_g), MASW_EALIGN,
               "draft_boundary_attend: slot inputs must be 16-byte aligned");
  MASW_REQUIRE(mem->slots_upper < mem->cfg.max_slots, MASW_ECAPACITY, "draft_boundary_attend: slot region full (%d slots)",
               mem->cfg.max_slots);
  SlotInputs slot;
  slot.h_g = h_g; slot.Wk_g = Wk_g; slot.Wv_g = Wv_g; slot.slot_pos = slot_pos; slot.active = active;
  return draft_attend_impl(mem, layer, k_raw, v_raw, slot, q, n_q, 1, o, lse, o_bf16, stream, "draft_boundary_attend");
}

extern "C" size_t verify_workspace_bytes(const masw_kv_desc* kv, int T) {
  if (kv == nullptr || T < 1 || kv->n_kv_heads < 1 || kv->n_q_heads % kv->n_kv_heads != 0) return 0;
  return verify_ws(kv->batch, kv->n_kv_heads, kv->n_q_heads / kv->n_kv_heads, kv->head_dim, T).total;
}

extern "C" int verify_attend(const masw_kv_desc* kv, const void* q, int T, float* o, float* lse, void* o_bf16,
                             void* workspace, size_t workspace_bytes, void* stream) {
  MASW_REQUIRE(kv != nullptr && q != nullptr && o != nullptr && workspace != nullptr, MASW_EINVAL, "verify_attend: null argument");
  MASW_REQUIRE(kv->k != nullptr && kv->v != nullptr && kv->kv_len != nullptr, MASW_EINVAL, "verify_attend: null cache pointer");
  MASW_REQUIRE(kv->head_dim == 64 || kv->head_dim == 128, MASW_EINVAL, "verify_attend: head_dim must be 64 or 128");
  MASW_REQUIRE(kv->batch >= 1 && kv->n_kv_heads >= 1 && kv->n_q_heads >= kv->n_kv_heads &&
                   kv->n_q_heads % kv->n_kv_heads == 0 && kv->capacity >= 1,
               MASW_EINVAL, "verify_attend: bad cache geometry");
  const int G = kv->n_q_heads / kv->n_kv_heads;
  MASW_REQUIRE(T >= 1 && T * G <= 64, MASW_EINVAL, "verify_attend: T * group size = %d exceeds 64", T * G);
  MASW_REQUIRE(aligned16(kv->k) && aligned16(kv->v) && aligned16(q) && aligned16(o) && aligned16(o_bf16) && aligned16(workspace),
               MASW_EALIGN, "verify_attend: pointers must be 16-byte aligned");
  MASW_REQUIRE(kv->stride_n % 8 == 0 && kv->stride_h % 8 == 0 && kv->stride_b % 8 == 0 && kv->stride_n >= kv->head_dim,
               MASW_EALIGN, "verify_attend: strides must be multiples of 8 elements and stride_n >= head_dim");
  const VerifyWs w = verify_ws(kv->batch, kv->n_kv_heads, G, kv->head_dim, T);
  MASW_REQUIRE(workspace_bytes >= w.total, MASW_ECAPACITY, "verify_attend: workspace %zu < %zu bytes", workspace_bytes, w.total);
  const int mt = (T * G + 15) / 16;
  const bool use_tc = (kv->head_dim == 128);
  CUtensorMap tk, tv;
  int rc = get_kv_maps(*kv, use_tc ? 128 : tile_entries(kv->head_dim, mt), &tk, &tv);
  if (rc != MASW_OK) return rc;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  AttendParams p{};
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.o = o; p.lse = lse; p.o_bf16 = static_cast<__nv_bfloat16*>(o_bf16);
  p.part_o = reinterpret_cast<unsigned long long*>(ws + w.off_part_o);
  p.part_ml = reinterpret_cast<unsigned long long*>(ws + w.off_part_ml);
  p.tickets = reinterpret_cast<int*>(ws + w.off_tickets);
  p.status = kv->status;
  p.deterministic = (kv->flags & MASW_KV_DETERMINISTIC) ? 1 : 0;
  p.early = (kv->flags & MASW_KV_STABLE) ? 1 : 0;
  p.t = nullptr; p.n_slots = nullptr; p.kv_len = kv->kv_len;
  p.n_q = T; p.last_row_is_slot = 0;
  p.G = G; p.Hq = kv->n_q_heads; p.Hkv = kv->n_kv_heads;
  p.S = 0; p.W = 0; p.ring_cap = 1; p.max_slots = 0;
  p.capacity = kv->capacity;
  const float scale = kv->softmax_scale > 0.f ? kv->softmax_scale : 1.0f / sqrtf(static_cast<float>(kv->head_dim));
  p.scale_log2e = scale * 1.4426950408889634f;
  if (use_tc) {
    const int tiles_upper = (kv->capacity + 127) / 128;
    // the next call's cache (an L2 hint): its tensor maps, or this call's own when there is none (never used then)
    CUtensorMap tkn = tk, tvn = tv;
    p.next_hint = 0;
    if (kv->next_k != nullptr && kv->next_v != nullptr && aligned16(kv->next_k) && aligned16(kv->next_v)) {
      masw_kv_desc nx = *kv;
      nx.k = kv->next_k; nx.v = kv->next_v;
      rc = get_kv_maps(nx, 128, &tkn, &tvn);
      if (rc != MASW_OK) return rc;
      p.next_hint = 1;
    }
    if (T * G <= 32)
      return launch_attend_tc<32, 3, 3>(tk, tv, tkn, tvn, p, kv->batch, kv->n_kv_heads, tiles_upper, w.splits_max, static_cast<cudaStream_t>(stream));
    return launch_attend_tc<64, 2, 3>(tk, tv, tkn, tvn, p, kv->batch, kv->n_kv_heads, tiles_upper, w.splits_max, static_cast<cudaStream_t>(stream));
  }
  return dispatch_attend(kv->head_dim, mt, tk, tv, p, kv->batch, kv->n_kv_heads, kv->capacity, 1, w.splits_max,
                         static_cast<cudaStream_t>(stream));
}

extern "C" size_t verify_paged_workspace_bytes(const masw_paged_kv_desc* kv, int T) {
  if (kv == nullptr || T < 1 || kv->n_kv_heads < 1 || kv->n_q_heads % kv->n_kv_heads != 0) return 0;
  return verify_ws(kv->batch, kv->n_kv_heads, kv->n_q_heads / kv->n_kv_heads, kv->head_dim, T).total;
}

extern "C" int verify_attend_paged(const masw_paged_kv_desc* kv, const void* q, int T, float* o, float* lse, void* o_bf16,
                                   void* workspace, size_t workspace_bytes, void* stream) {
  MASW_REQUIRE(kv != nullptr && q != nullptr && o != nullptr && workspace != nullptr, MASW_EINVAL,
               "verify_attend_paged: null argument");
  MASW_REQUIRE(kv->k_pages != nullptr && kv->v_pages != nullptr && kv->page_table != nullptr && kv->kv_len != nullptr,
               MASW_EINVAL, "verify_attend_paged: null cache pointer");
  MASW_REQUIRE(kv->head_dim == 128, MASW_EINVAL, "verify_attend_paged: head_dim must be 128");
  MASW_REQUIRE(kv->batch >= 1 && kv->n_kv_heads >= 1 && kv->n_q_heads >= kv->n_kv_heads &&
                   kv->n_q_heads % kv->n_kv_heads == 0 && kv->n_pages >= 1 && kv->max_pages >= 1,
               MASW_EINVAL, "verify_attend_paged: bad cache geometry");
  const int G = kv->n_q_heads / kv->n_kv_heads;
  MASW_REQUIRE(T >= 1 && T * G <= 64, MASW_EINVAL, "verify_attend_paged: T * group size = %d exceeds 64", T * G);
  MASW_REQUIRE(aligned16(kv->k_pages) && aligned16(kv->v_pages) && aligned16(q) && aligned16(o) && aligned16(o_bf16) &&
                   aligned16(workspace),
               MASW_EALIGN, "verify_attend_paged: pointers must be 16-byte aligned");
  const VerifyWs w = verify_ws(kv->batch, kv->n_kv_heads, G, kv->head_dim, T);
  MASW_REQUIRE(workspace_bytes >= w.total, MASW_ECAPACITY, "verify_attend_paged: workspace %zu < %zu bytes", workspace_bytes,
               w.total);
  // the pool as a 4-D tensor: (head_dim, 128 entries of a page, kv head, page)
  masw_kv_desc pool{};
  pool.k = kv->k_pages; pool.v = kv->v_pages;
  pool.stride_n = kv->head_dim;
  pool.stride_h = static_cast<int64_t>(128) * kv->head_dim;
  pool.stride_b = pool.stride_h * kv->n_kv_heads;
  pool.batch = kv->n_pages; pool.n_q_heads = kv->n_q_heads; pool.n_kv_heads = kv->n_kv_heads; pool.head_dim = kv->head_dim;
  pool.capacity = 128;
  CUtensorMap tk, tv;
  int rc = get_kv_maps(pool, 128, &tk, &tv);
  if (rc != MASW_OK) return rc;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  AttendParams p{};
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.o = o; p.lse = lse; p.o_bf16 = static_cast<__nv_bfloat16*>(o_bf16);
  p.part_o = reinterpret_cast<unsigned long long*>(ws + w.off_part_o);
  p.part_ml = reinterpret_cast<unsigned long long*>(ws + w.off_part_ml);
  p.tickets = reinterpret_cast<int*>(ws + w.off_tickets);
  p.status = kv->status;
  p.deterministic = (kv->flags & MASW_KV_DETERMINISTIC) ? 1 : 0;
  p.t = nullptr; p.n_slots = nullptr; p.kv_len = kv->kv_len;
  p.n_q = T; p.last_row_is_slot = 0;
  p.G = G; p.Hq = kv->n_q_heads; p.Hkv = kv->n_kv_heads;
  p.S = 0; p.W = 0; p.ring_cap = 1; p.max_slots = 0;
  p.capacity = kv->max_pages * 128;
  p.page_table = kv->page_table;
  p.max_pages = kv->max_pages;
  const float scale = kv->softmax_scale > 0.f ? kv->softmax_scale : 1.0f / sqrtf(static_cast<float>(kv->head_dim));
  p.scale_log2e = scale * 1.4426950408889634f;
  if (T * G <= 32)
    return launch_attend_tc<32, 3, 3>(tk, tv, tk, tv, p, kv->batch, kv->n_kv_heads, kv->max_pages, w.splits_max, static_cast<cudaStream_t>(stream));
  return launch_attend_tc<64, 2, 3>(tk, tv, tk, tv, p, kv->batch, kv->n_kv_heads, kv->max_pages, w.splits_max, static_cast<cudaStream_t>(stream));
}


// ---- verify_attend_fp8: the verifier's attention over a paged e4m3 cache ---------------------------------
extern "C" size_t verify_fp8_workspace_bytes(const masw_fp8_kv_desc* kv, int T) {
  if (kv == nullptr || T < 1 || kv->n_kv_heads < 1 || kv->n_q_heads % kv->n_kv_heads != 0) return 0;
  return verify_ws(kv->batch, kv->n_kv_heads, kv->n_q_heads / kv->n_kv_heads, kv->head_dim, T).total;
}

extern "C" int verify_attend_fp8(const masw_fp8_kv_desc* kv, const void* q, int T, float* o, float* lse, void* o_bf16,
                                 void* workspace, size_t workspace_bytes, void* stream) {
  MASW_REQUIRE(kv != nullptr && q != nullptr && o != nullptr && workspace != nullptr, MASW_EINVAL,
               "verify_attend_fp8: null argument");
  MASW_REQUIRE(kv->k_pages != nullptr && kv->v_pages != nullptr && kv->k_scale != nullptr && kv->v_scale != nullptr &&
                   kv->page_table != nullptr && kv->kv_len != nullptr,
               MASW_EINVAL, "verify_attend_fp8: null cache pointer");
  MASW_REQUIRE(kv->head_dim == 128, MASW_EINVAL, "verify_attend_fp8: head_dim must be 128");
  MASW_REQUIRE(kv->batch >= 1 && kv->n_kv_heads >= 1 && kv->n_q_heads >= kv->n_kv_heads &&
                   kv->n_q_heads % kv->n_kv_heads == 0 && kv->n_pages >= 1 && kv->max_pages >= 1,
               MASW_EINVAL, "verify_attend_fp8: bad cache geometry");
  const int G = kv->n_q_heads / kv->n_kv_heads;
  MASW_REQUIRE(T >= 1 && T * G <= 32, MASW_EINVAL, "verify_attend_fp8: T * group size = %d exceeds 32", T * G);
  MASW_REQUIRE(aligned16(kv->k_pages) && aligned16(kv->v_pages) && aligned16(q) && aligned16(o) && aligned16(o_bf16) &&
                   aligned16(workspace),
               MASW_EALIGN, "verify_attend_fp8: pointers must be 16-byte aligned");
  const VerifyWs w = verify_ws(kv->batch, kv->n_kv_heads, G, kv->head_dim, T);
  MASW_REQUIRE(workspace_bytes >= w.total, MASW_ECAPACITY, "verify_attend_fp8: workspace %zu < %zu bytes", workspace_bytes,
               w.total);
  CUtensorMap tk, tv;
  int rc = encode_fp8_page_map(&tk, kv->k_pages, kv->n_kv_heads, kv->n_pages);
  if (rc != MASW_OK) return rc;
  rc = encode_fp8_page_map(&tv, kv->v_pages, kv->n_kv_heads, kv->n_pages);
  if (rc != MASW_OK) return rc;
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  AttendParams p{};
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.o = o; p.lse = lse; p.o_bf16 = static_cast<__nv_bfloat16*>(o_bf16);
  p.part_o = reinterpret_cast<unsigned long long*>(ws + w.off_part_o);
  p.part_ml = reinterpret_cast<unsigned long long*>(ws + w.off_part_ml);
  p.tickets = reinterpret_cast<int*>(ws + w.off_tickets);
  p.status = kv->status;
  p.deterministic = (kv->flags & MASW_KV_DETERMINISTIC) ? 1 : 0;
  p.kv_len = kv->kv_len;
  p.n_q = T; p.last_row_is_slot = 0;
  p.G = G; p.Hq = kv->n_q_heads; p.Hkv = kv->n_kv_heads;
  p.S = 0; p.W = 0; p.ring_cap = 1; p.max_slots = 0;
  p.capacity = kv->max_pages * 128;
  p.page_table = kv->page_table;
  p.max_pages = kv->max_pages;
  p.k_scale = kv->k_scale; p.v_scale = kv->v_scale;
  const float scale = kv->softmax_scale > 0.f ? kv->softmax_scale : 1.0f / sqrtf(static_cast<float>(kv->head_dim));
  p.scale_log2e = scale * 1.4426950408889634f;
  // one K operand buffer (free again as soon as S^T is computed), two V operand buffers, three raw tiles per ring
  return launch_attend_tc<32, 1, 2, true>(tk, tv, tk, tv, p, kv->batch, kv->n_kv_heads, kv->max_pages, w.splits_max,
                                          static_cast<cudaStream_t>(stream));
}
