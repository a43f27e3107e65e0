// draft_prefill_attend: the draft's masked prefill pass of one layer (Section 4.3 "Prefill", Appendix C).
#include <algorithm>
#include <cmath>

#include "mem_handle.cuh"
#include "prefill_tc_kernel.cuh"

namespace masw {

template <int D, int NS, int NK, int NV>
static int launch_prefill(const CUtensorMap& tmK, const CUtensorMap& tmV, PrefillParams p, int B, cudaStream_t st) {
  using C = PrefillCfg<D, NS, NK, NV>;
  auto kern = prefill_tc_kernel<D, NS, NK, NV>;
  p.n_raw_tiles = (p.P + NS * p.T - 1) / (NS * p.T);
  p.n_slot_tiles = (p.M + NS * p.T - 1) / (NS * p.T);
  static bool configured = false;
  if (!configured) {
    MASW_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, C::kSmemBytes));
    configured = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.n_raw_tiles + p.n_slot_tiles, p.Hkv, B);
  cfg.blockDim = dim3(C::kThreads, 1, 1);
  cfg.dynamicSmemBytes = C::kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  MASW_CUDA_TRY(cudaLaunchKernelEx(&cfg, kern, tmK, tmV, p));
  count_launch();
  return MASW_OK;
}

}  // namespace masw

using namespace masw;

extern "C" int draft_prefill_slots(const masw_config* cfg, int P) {
  if (cfg == nullptr || P < 0 || cfg->slot_interval < 1) return -1;
  return P > cfg->sink ? (P - cfg->sink) / cfg->slot_interval : 0;
}

extern "C" int draft_prefill_attend(masw_mem* mem, int layer, const masw_kv_desc* kv, const void* q, int P, float* o,
                                    float* lse, void* o_bf16, int import_memory, void* stream) {
  MASW_REQUIRE(mem != nullptr && kv != nullptr && q != nullptr, MASW_EINVAL, "draft_prefill_attend: null argument");
  { const int rc = flush_counters(mem, static_cast<cudaStream_t>(stream)); if (rc != MASW_OK) return rc; }
  mem->kv_clean = false;   // the import writes the arena
  MASW_REQUIRE(o != nullptr || o_bf16 != nullptr, MASW_EINVAL, "draft_prefill_attend: one of o, o_bf16 must be given");
  MASW_REQUIRE(kv->k != nullptr && kv->v != nullptr, MASW_EINVAL, "draft_prefill_attend: null K/V pointer");
  const masw_config& c = mem->cfg;
  MASW_REQUIRE(layer >= 0 && layer < c.n_layers, MASW_EINVAL, "draft_prefill_attend: layer %d out of range", layer);
  MASW_REQUIRE(kv->batch == c.batch && kv->n_q_heads == c.n_q_heads && kv->n_kv_heads == c.n_kv_heads &&
                   kv->head_dim == c.head_dim,
               MASW_EINVAL, "draft_prefill_attend: K/V geometry differs from the memory's configuration");
  MASW_REQUIRE(P >= 1, MASW_EINVAL, "draft_prefill_attend: empty prefix");
  const int M = draft_prefill_slots(&c, P);
  MASW_REQUIRE(M <= c.max_slots, MASW_ECAPACITY, "draft_prefill_attend: %d slots exceed max_slots = %d", M, c.max_slots);
  MASW_REQUIRE(kv->capacity >= P + M, MASW_ECAPACITY, "draft_prefill_attend: K/V hold %d entries, %d needed (P + slots)",
               kv->capacity, P + M);
  const int G = c.n_q_heads / c.n_kv_heads;
  MASW_REQUIRE(G >= 1 && G <= 128 && 128 % G == 0, MASW_EINVAL, "draft_prefill_attend: group size %d must divide 128", G);
  MASW_REQUIRE(aligned16(kv->k) && aligned16(kv->v) && aligned16(q) && aligned16(o) && aligned16(o_bf16), MASW_EALIGN,
               "draft_prefill_attend: pointers must be 16-byte aligned");
  MASW_REQUIRE(kv->stride_n % 8 == 0 && kv->stride_h % 8 == 0 && kv->stride_b % 8 == 0 && kv->stride_n >= kv->head_dim,
               MASW_EALIGN, "draft_prefill_attend: strides must be multiples of 8 elements and stride_n >= head_dim");
  CUtensorMap tk, tv;
  int rc = get_kv_maps(*kv, 128, &tk, &tv);
  if (rc != MASW_OK) return rc;
  PrefillParams p{};
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.o = o; p.lse = lse; p.o_bf16 = static_cast<__nv_bfloat16*>(o_bf16);
  p.status = mem->d_status;
  p.P = P; p.M = M; p.S = c.sink; p.W = c.window; p.r = c.slot_interval;
  p.G = G; p.Hq = c.n_q_heads; p.Hkv = c.n_kv_heads;
  p.T = 128 / G;
  p.scale_log2e = mem->scale * 1.4426950408889634f;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  rc = (c.head_dim == 64) ? launch_prefill<64, 2, 3, 3>(tk, tv, p, c.batch, st) : launch_prefill<128, 1, 2, 2>(tk, tv, p, c.batch, st);
  if (rc != MASW_OK) return rc;
  if (import_memory) {
    // the memory the pass has built: sinks, every slot, and the raw tokens the ring retains behind position P
    const int64_t strides[3] = {kv->stride_b, kv->stride_n, kv->stride_h};
    const __nv_bfloat16* k = static_cast<const __nv_bfloat16*>(kv->k);
    const __nv_bfloat16* v = static_cast<const __nv_bfloat16*>(kv->v);
    const int n_sink = std::min(c.sink, P);
    if (n_sink > 0) {
      rc = mem_load(mem, layer, MASW_REGION_SINK, k, v, 0, n_sink, strides, stream);
      if (rc != MASW_OK) return rc;
    }
    if (M > 0) {
      rc = mem_load(mem, layer, MASW_REGION_SLOT, k + static_cast<int64_t>(P) * kv->stride_n,
                    v + static_cast<int64_t>(P) * kv->stride_n, 0, M, strides, stream);
      if (rc != MASW_OK) return rc;
    }
    const int n_local = std::min(std::max(P - c.sink, 0), c.window + c.rollback);
    if (n_local > 0) {
      const int first = P - n_local;
      rc = mem_load(mem, layer, MASW_REGION_LOCAL, k + static_cast<int64_t>(first) * kv->stride_n,
                    v + static_cast<int64_t>(first) * kv->stride_n, first, n_local, strides, stream);
      if (rc != MASW_OK) return rc;
    }
  }
  return MASW_OK;
}
