// The draft's three-part KV memory: creation, prefill import, per-step update (raw-token append and
// memory-slot materialisation through the mirrored projections), counter advance and rollback.
#include <algorithm>
#include <cmath>
#include <new>

#include "mem_handle.cuh"

namespace masw {

struct MemGeom {
  int B, Hkv, D, S, max_slots, ring_cap, n_cap;
};

__device__ __forceinline__ size_t entry_offset(const MemGeom& g, int b, int h, int entry) {
  return ((static_cast<size_t>(b) * g.Hkv + h) * g.n_cap + entry) * g.D;
}

// entry index of raw token `pos`: sink region while pos < S, else the ring
__device__ __forceinline__ int raw_entry(const MemGeom& g, int pos) {
  return pos < g.S ? pos : g.S + g.max_slots + (pos - g.S) % g.ring_cap;
}

// (i) of mem_update: pending raw tokens t[b] .. t[b]+n_raw-1.  grid (n_raw, Hkv, B), D/8 threads.
__global__ void append_raw_kernel(__nv_bfloat16* K, __nv_bfloat16* V, const __nv_bfloat16* k_raw,
                                  const __nv_bfloat16* v_raw, const int* t, MemGeom g, int n_raw) {
  const int i = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int entry = raw_entry(g, t[b] + i);
  const size_t src = ((static_cast<size_t>(b) * n_raw + i) * g.Hkv + h) * g.D + threadIdx.x * 8;
  const size_t dst = entry_offset(g, b, h, entry) + threadIdx.x * 8;
  *reinterpret_cast<uint4*>(K + dst) = *reinterpret_cast<const uint4*>(k_raw + src);
  *reinterpret_cast<uint4*>(V + dst) = *reinterpret_cast<const uint4*>(v_raw + src);
}

// mem_load: strided import into one region.  grid (n, Hkv, B), D/8 threads.
__global__ void load_region_kernel(__nv_bfloat16* K, __nv_bfloat16* V, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                   MemGeom g, int region, int first, long long sb, long long sn, long long sh) {
  const int i = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  int entry;
  if (region == MASW_REGION_SINK) entry = first + i;
  else if (region == MASW_REGION_SLOT) entry = g.S + first + i;
  else entry = raw_entry(g, first + i);
  const size_t src = static_cast<size_t>(b * sb + i * sn + h * sh) + threadIdx.x * 8;
  const size_t dst = entry_offset(g, b, h, entry) + threadIdx.x * 8;
  *reinterpret_cast<uint4*>(K + dst) = *reinterpret_cast<const uint4*>(k + src);
  *reinterpret_cast<uint4*>(V + dst) = *reinterpret_cast<const uint4*>(v + src);
}

// (ii) of mem_update: K_g = RoPE(h_g W_K,g), V_g = h_g W_V,g for the pending slot of every active
// sequence.  grid (kProjKSplit, Hkv, 2): one CTA owns one head's D columns of W_K,g (z = 0) or W_V,g
// (z = 1) over one slice of the d_model rows.  The weights are streamed once with 16-byte loads,
// accumulated in fp32, reduced over the CTA, written as a k-split partial; the last CTA of the
// (head, K|V) to finish (atomic ticket) sums the partials in fixed order, rotates the key and stores
// bf16 at slot index n_slots[b].
constexpr int kProjThreads = 256;
constexpr int kProjBatchChunk = 4;

template <int D>
__global__ void __launch_bounds__(kProjThreads)
slot_project_kernel(__nv_bfloat16* K, __nv_bfloat16* V, const __nv_bfloat16* h_g, const __nv_bfloat16* Wk,
                    const __nv_bfloat16* Wv, const int* slot_pos, const uint8_t* active, const int* n_slots,
                    float* part, int* tickets, int* status, MemGeom g, int d_model, double rope_base) {
  constexpr int kColThreads = D / 8;
  constexpr int kLanes = kProjThreads / kColThreads;
  __shared__ float red[kLanes][kProjBatchChunk][D + 4];
  __shared__ float fin[D];
  __shared__ int last_flag;

  const int ks = blockIdx.x, h = blockIdx.y, kv = blockIdx.z;
  const int tid = threadIdx.x;
  const int ct = tid % kColThreads, kl = tid / kColThreads;
  const __nv_bfloat16* Wm = kv == 0 ? Wk : Wv;
  const int ncols = g.Hkv * D;
  const int rows_per = (d_model + kProjKSplit - 1) / kProjKSplit;
  const int k0 = ks * rows_per, k1 = min(d_model, k0 + rows_per);
  const size_t out_cols = static_cast<size_t>(2) * ncols;  // partial row: [K cols | V cols]

  for (int b0 = 0; b0 < g.B; b0 += kProjBatchChunk) {
    const int nb = min(kProjBatchChunk, g.B - b0);
    float acc[kProjBatchChunk][8];
#pragma unroll
    for (int bb = 0; bb < kProjBatchChunk; ++bb)
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[bb][c] = 0.f;
    for (int k = k0 + kl; k < k1; k += kLanes) {
      const uint4 w4 = __ldg(reinterpret_cast<const uint4*>(Wm + static_cast<size_t>(k) * ncols + h * D + ct * 8));
      const __nv_bfloat162* w2 = reinterpret_cast<const __nv_bfloat162*>(&w4);
      float w[8];
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const float2 f = __bfloat1622float2(w2[c]);
        w[2 * c] = f.x; w[2 * c + 1] = f.y;
      }
#pragma unroll
      for (int bb = 0; bb < kProjBatchChunk; ++bb) {
        if (bb < nb) {
          const float x = __bfloat162float(h_g[static_cast<size_t>(b0 + bb) * d_model + k]);
#pragma unroll
          for (int c = 0; c < 8; ++c) acc[bb][c] = fmaf(x, w[c], acc[bb][c]);
        }
      }
    }
#pragma unroll
    for (int bb = 0; bb < kProjBatchChunk; ++bb)
#pragma unroll
      for (int c = 0; c < 8; ++c) red[kl][bb][ct * 8 + c] = acc[bb][c];
    __syncthreads();
    for (int idx = tid; idx < nb * D; idx += kProjThreads) {
      const int bb = idx / D, col = idx % D;
      float sum = 0.f;
      for (int l = 0; l < kLanes; ++l) sum += red[l][bb][col];
      part[(static_cast<size_t>(ks) * g.B + b0 + bb) * out_cols + kv * ncols + h * D + col] = sum;
    }
    __syncthreads();
  }

  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int ticket = atomicAdd(&tickets[kv * g.Hkv + h], 1);
    last_flag = (ticket == kProjKSplit - 1) ? 1 : 0;
  }
  __syncthreads();
  if (last_flag == 0) return;
  __threadfence();

  __nv_bfloat16* dst_base = kv == 0 ? K : V;
  for (int b = 0; b < g.B; ++b) {
    if (active != nullptr && active[b] == 0) continue;   // uniform across the CTA
    const int m = n_slots[b];
    if (m >= g.max_slots) {
      if (tid == 0 && status) atomicOr(status, MASW_STATUS_SLOT_OVERFLOW);
      continue;
    }
    if (tid < D) {
      float sum = 0.f;
      for (int s = 0; s < kProjKSplit; ++s)
        sum += __ldcg(part + (static_cast<size_t>(s) * g.B + b) * out_cols + kv * ncols + h * D + tid);
      fin[tid] = sum;
    }
    __syncthreads();
    if (tid < D) {
      float val = fin[tid];
      if (kv == 0) {
        // rotate-half pairing (i, i + D/2), angle pos * base^(-2i/D), evaluated in double
        const int i = tid % (D / 2);
        const double theta = static_cast<double>(slot_pos[b]) * pow(rope_base, -2.0 * i / D);
        double sn, cs;
        sincos(theta, &sn, &cs);
        const double x1 = fin[i], x2 = fin[i + D / 2];
        val = static_cast<float>(tid < D / 2 ? x1 * cs - x2 * sn : x2 * cs + x1 * sn);
      }
      dst_base[entry_offset(g, b, h, g.S + m) + tid] = __float2bfloat16_rn(val);
    }
    __syncthreads();
  }
  if (tid == 0) tickets[kv * g.Hkv + h] = 0;
}

__global__ void advance_kernel(int* t, int* n_slots, int* status, const uint8_t* active, int B, int n_tokens,
                               int add_slot, int max_slots) {
  // Launched with programmatic stream serialisation: the next launch (an attention layer, which reads the
  // counters only behind its own wait) may be set up at once, and the counters are written only when the
  // launch in front of this one, which still reads them, has completed.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  t[b] += n_tokens;
  if (add_slot && (active == nullptr || active[b] != 0)) {   // add_slot: how many slots were committed (one, or several deferred)
    const int m = n_slots[b] + add_slot;
    n_slots[b] = min(m, max_slots);
    if (m > max_slots && status) atomicOr(status, MASW_STATUS_SLOT_OVERFLOW);
  }
}

__global__ void rollback_kernel(int* t, int* n_slots, const int* t_keep, const int* slots_keep, int B, int pend_t, int pend_m,
                                int max_slots) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // as in advance_kernel
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  // (pend_t, pend_m): a deferred counter update that this launch applies on the way
  t[b] = max(0, min(t[b] + pend_t, t_keep[b]));
  n_slots[b] = max(0, min(min(n_slots[b] + pend_m, max_slots), slots_keep[b]));
}

static int validate_config(const masw_config* c) {
  MASW_REQUIRE(c != nullptr, MASW_EINVAL, "null config");
  MASW_REQUIRE(c->n_layers >= 1 && c->batch >= 1, MASW_EINVAL, "n_layers and batch must be >= 1");
  MASW_REQUIRE(c->head_dim == 64 || c->head_dim == 128, MASW_EINVAL, "head_dim must be 64 or 128, got %d", c->head_dim);
  MASW_REQUIRE(c->n_kv_heads >= 1 && c->n_q_heads >= c->n_kv_heads && c->n_q_heads % c->n_kv_heads == 0, MASW_EINVAL,
               "n_q_heads must be a multiple of n_kv_heads");
  MASW_REQUIRE(c->d_model >= 8 && c->d_model % 8 == 0, MASW_EINVAL, "d_model must be a positive multiple of 8");
  MASW_REQUIRE(c->sink >= 0 && c->window >= 1 && c->slot_interval >= 1 && c->rollback >= 0 && c->max_slots >= 0,
               MASW_EINVAL, "sink/window/slot_interval/rollback/max_slots out of range");
  MASW_REQUIRE(c->gamma_max >= 1, MASW_EINVAL, "gamma_max must be >= 1");
  MASW_REQUIRE((c->gamma_max + 1) * (c->n_q_heads / c->n_kv_heads) <= 64, MASW_EINVAL,
               "(gamma_max + 1) * group size must be <= 64");
  MASW_REQUIRE(c->softmax_scale >= 0.f && c->rope_base >= 0.f, MASW_EINVAL, "softmax_scale and rope_base must be >= 0");
  return MASW_OK;
}

static MemGeom geom_of(const masw_mem* m) {
  return MemGeom{m->cfg.batch, m->cfg.n_kv_heads, m->cfg.head_dim, m->cfg.sink, m->cfg.max_slots, m->ring_cap, m->n_cap};
}

// The counter kernels let their successor be set up early only where that pays: the successor's CTAs then sit
// beside the still running attention launch, and at large batch (a bandwidth- and issue-bound launch of hundreds
// of MB) that cost 5 % of the launch, while a batch-1 decode step gains a little.  Same size rule as the
// attention launch's own early L2 hint.
static int counters_overlap(const masw_mem* m) {
  const masw_config& c = m->cfg;
  const long long entries = c.sink + std::min(m->slots_upper + 1, c.max_slots) + c.window;
  return (4LL * entries * c.batch * c.n_kv_heads * c.head_dim <= (48LL << 20)) ? 1 : 0;
}

static int launch_advance(masw_mem* mem, int n_tokens, int add_slots, const uint8_t* active, cudaStream_t st) {
  const int B = mem->cfg.batch;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((B + 127) / 128, 1, 1);
  cfg.blockDim = dim3(128, 1, 1);
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = counters_overlap(mem);
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  MASW_CUDA_TRY(cudaLaunchKernelEx(&cfg, advance_kernel, mem->d_t, mem->d_slots, mem->d_status, active, B, n_tokens, add_slots,
                                   mem->cfg.max_slots));
  count_launch();
  return MASW_OK;
}

int flush_counters(masw_mem* mem, cudaStream_t st) {
  if (mem->pend_t == 0 && mem->pend_m == 0) return MASW_OK;
  const int dt = mem->pend_t, dm = mem->pend_m;
  mem->pend_t = 0;
  mem->pend_m = 0;
  mem->kv_clean = false;   // the counters are written: the next attention launch reads them behind its wait
  return launch_advance(mem, dt, dm, nullptr, st);
}

}  // namespace masw

using namespace masw;

extern "C" int masw_sizes(const masw_config* cfg, size_t* kv_arena_bytes, size_t* workspace_bytes) {
  int rc = validate_config(cfg);
  if (rc != MASW_OK) return rc;
  const size_t per_tensor = static_cast<size_t>(cfg->batch) * cfg->n_kv_heads * entries_per_head(*cfg) * cfg->head_dim * 2;
  if (kv_arena_bytes) *kv_arena_bytes = per_tensor * 2 * cfg->n_layers;
  if (workspace_bytes) *workspace_bytes = ws_layout(*cfg).total;
  return MASW_OK;
}

extern "C" int mem_init(const masw_config* cfg, void* kv_arena, size_t kv_arena_bytes, void* workspace,
                        size_t workspace_bytes, void* stream, masw_mem** out) {
  int rc = validate_config(cfg);
  if (rc != MASW_OK) return rc;
  MASW_REQUIRE(kv_arena != nullptr && workspace != nullptr && out != nullptr, MASW_EINVAL, "mem_init: null argument");
  MASW_REQUIRE((reinterpret_cast<uintptr_t>(kv_arena) & 255) == 0 && (reinterpret_cast<uintptr_t>(workspace) & 255) == 0,
               MASW_EALIGN, "mem_init: arena and workspace must be 256-byte aligned");
  size_t need_arena = 0, need_ws = 0;
  masw_sizes(cfg, &need_arena, &need_ws);
  MASW_REQUIRE(kv_arena_bytes >= need_arena, MASW_ECAPACITY, "mem_init: arena %zu < %zu bytes", kv_arena_bytes, need_arena);
  MASW_REQUIRE(workspace_bytes >= need_ws, MASW_ECAPACITY, "mem_init: workspace %zu < %zu bytes", workspace_bytes, need_ws);
  int ndev = 0;
  MASW_CUDA_TRY(cudaGetDeviceCount(&ndev));
  MASW_REQUIRE(ndev > 0, MASW_ECUDA, "mem_init: no CUDA device");

  masw_mem* m = new (std::nothrow) masw_mem();
  MASW_REQUIRE(m != nullptr, MASW_EINVAL, "mem_init: out of host memory");
  m->cfg = *cfg;
  m->G = cfg->n_q_heads / cfg->n_kv_heads;
  m->ring_cap = ring_capacity(*cfg);
  m->n_cap = entries_per_head(*cfg);
  m->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / sqrtf(static_cast<float>(cfg->head_dim));
  m->rope_base = cfg->rope_base > 0.f ? static_cast<double>(cfg->rope_base) : 500000.0;
  m->arena = static_cast<uint8_t*>(kv_arena);
  m->arena_bytes = need_arena;
  m->tensor_elems = static_cast<size_t>(cfg->batch) * cfg->n_kv_heads * m->n_cap * cfg->head_dim;
  m->ws = static_cast<uint8_t*>(workspace);
  m->L = ws_layout(*cfg);
  m->d_t = reinterpret_cast<int*>(m->ws + m->L.off_t);
  m->d_slots = reinterpret_cast<int*>(m->ws + m->L.off_slots);
  m->d_status = reinterpret_cast<int*>(m->ws + m->L.off_status);
  m->d_tickets_attn = reinterpret_cast<int*>(m->ws + m->L.off_tickets_attn);
  m->d_tickets_proj = reinterpret_cast<int*>(m->ws + m->L.off_tickets_proj);
  m->d_part_o = reinterpret_cast<unsigned long long*>(m->ws + m->L.off_part_o);
  m->d_part_ml = reinterpret_cast<unsigned long long*>(m->ws + m->L.off_part_ml);
  m->d_proj_part = reinterpret_cast<float*>(m->ws + m->L.off_proj_part);
  m->d_part_slot = reinterpret_cast<unsigned long long*>(m->ws + m->L.off_part_slot);
  m->slots_upper = 0;
  m->tmK32.resize(cfg->n_layers); m->tmV32.resize(cfg->n_layers);
  m->tmK64.resize(cfg->n_layers); m->tmV64.resize(cfg->n_layers);
  const int64_t sn = cfg->head_dim, sh = static_cast<int64_t>(m->n_cap) * cfg->head_dim,
                sb = sh * cfg->n_kv_heads;
  for (int l = 0; l < cfg->n_layers && rc == MASW_OK; ++l) {
    rc = encode_kv_tensor_map(&m->tmK32[l], m->k_layer(l), cfg->head_dim, m->n_cap, cfg->n_kv_heads, cfg->batch, sn, sh, sb, 32);
    if (rc == MASW_OK) rc = encode_kv_tensor_map(&m->tmV32[l], m->v_layer(l), cfg->head_dim, m->n_cap, cfg->n_kv_heads, cfg->batch, sn, sh, sb, 32);
    if (rc == MASW_OK) rc = encode_kv_tensor_map(&m->tmK64[l], m->k_layer(l), cfg->head_dim, m->n_cap, cfg->n_kv_heads, cfg->batch, sn, sh, sb, 64);
    if (rc == MASW_OK) rc = encode_kv_tensor_map(&m->tmV64[l], m->v_layer(l), cfg->head_dim, m->n_cap, cfg->n_kv_heads, cfg->batch, sn, sh, sb, 64);
  }
  if (rc == MASW_OK) rc = check_cuda(cudaMemsetAsync(m->arena, 0, need_arena, static_cast<cudaStream_t>(stream)), "zero arena");
  if (rc == MASW_OK) rc = check_cuda(cudaMemsetAsync(m->ws, 0, m->L.total, static_cast<cudaStream_t>(stream)), "zero workspace");
  if (rc != MASW_OK) { delete m; return rc; }
  *out = m;
  return MASW_OK;
}

extern "C" void mem_free(masw_mem* mem) { delete mem; }

extern "C" int mem_load(masw_mem* mem, int layer, int region, const void* k, const void* v, int first, int n,
                        const int64_t strides[3], void* stream) {
  MASW_REQUIRE(mem != nullptr && k != nullptr && v != nullptr && strides != nullptr, MASW_EINVAL, "mem_load: null argument");
  { const int rc = flush_counters(mem, static_cast<cudaStream_t>(stream)); if (rc != MASW_OK) return rc; }
  mem->kv_clean = false;   // this call writes the counters or the arena: the next attention launch reads them behind its wait
  MASW_REQUIRE(layer >= 0 && layer < mem->cfg.n_layers, MASW_EINVAL, "mem_load: layer %d out of range", layer);
  MASW_REQUIRE(n >= 0 && first >= 0, MASW_EINVAL, "mem_load: negative count or index");
  MASW_REQUIRE(aligned16(k) && aligned16(v), MASW_EALIGN, "mem_load: pointers must be 16-byte aligned");
  MASW_REQUIRE(strides[0] % 8 == 0 && strides[1] % 8 == 0 && strides[2] % 8 == 0, MASW_EALIGN,
               "mem_load: strides must be multiples of 8 elements");
  const masw_config& c = mem->cfg;
  if (region == MASW_REGION_SINK) {
    MASW_REQUIRE(first + n <= c.sink, MASW_ECAPACITY, "mem_load: sink range [%d, %d) exceeds S = %d", first, first + n, c.sink);
  } else if (region == MASW_REGION_SLOT) {
    MASW_REQUIRE(first + n <= c.max_slots, MASW_ECAPACITY, "mem_load: slot range [%d, %d) exceeds max_slots = %d", first, first + n, c.max_slots);
  } else if (region == MASW_REGION_LOCAL) {
    MASW_REQUIRE(first >= c.sink, MASW_EINVAL, "mem_load: local positions start at S = %d", c.sink);
    MASW_REQUIRE(n <= mem->ring_cap, MASW_ECAPACITY, "mem_load: %d tokens exceed the ring of %d", n, mem->ring_cap);
  } else {
    MASW_REQUIRE(false, MASW_EINVAL, "mem_load: unknown region %d", region);
  }
  if (n == 0) return MASW_OK;
  dim3 grid(n, c.n_kv_heads, c.batch);
  load_region_kernel<<<grid, c.head_dim / 8, 0, static_cast<cudaStream_t>(stream)>>>(
      mem->k_layer(layer), mem->v_layer(layer), static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v),
      geom_of(mem), region, first, strides[0], strides[1], strides[2]);
  count_launch();
  MASW_CUDA_TRY(cudaGetLastError());
  return MASW_OK;
}

extern "C" int mem_set_state(masw_mem* mem, const int32_t* t, const int32_t* n_slots, void* stream) {
  MASW_REQUIRE(mem != nullptr, MASW_EINVAL, "mem_set_state: null handle");
  { const int rc = flush_counters(mem, static_cast<cudaStream_t>(stream)); if (rc != MASW_OK) return rc; }
  mem->kv_clean = false;   // this call writes the counters or the arena: the next attention launch reads them behind its wait
  const int B = mem->cfg.batch;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (t) {
    for (int b = 0; b < B; ++b) MASW_REQUIRE(t[b] >= 0, MASW_EINVAL, "mem_set_state: negative token count");
    MASW_CUDA_TRY(cudaMemcpyAsync(mem->d_t, t, sizeof(int) * B, cudaMemcpyHostToDevice, st));
  }
  if (n_slots) {
    int mx = 0;
    for (int b = 0; b < B; ++b) {
      MASW_REQUIRE(n_slots[b] >= 0 && n_slots[b] <= mem->cfg.max_slots, MASW_ECAPACITY,
                   "mem_set_state: slot count %d outside [0, %d]", n_slots[b], mem->cfg.max_slots);
      mx = std::max(mx, n_slots[b]);
    }
    MASW_CUDA_TRY(cudaMemcpyAsync(mem->d_slots, n_slots, sizeof(int) * B, cudaMemcpyHostToDevice, st));
    mem->slots_upper = mx;
  }
  return MASW_OK;
}

extern "C" int mem_get_state(masw_mem* mem, int32_t* t, int32_t* n_slots, int32_t* status, void* stream) {
  MASW_REQUIRE(mem != nullptr, MASW_EINVAL, "mem_get_state: null handle");
  { const int rc = flush_counters(mem, static_cast<cudaStream_t>(stream)); if (rc != MASW_OK) return rc; }
  const int B = mem->cfg.batch;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (t) MASW_CUDA_TRY(cudaMemcpyAsync(t, mem->d_t, sizeof(int) * B, cudaMemcpyDeviceToHost, st));
  if (n_slots) MASW_CUDA_TRY(cudaMemcpyAsync(n_slots, mem->d_slots, sizeof(int) * B, cudaMemcpyDeviceToHost, st));
  if (status) {   // the bits accumulate between reads: a read returns them and starts over
    MASW_CUDA_TRY(cudaMemcpyAsync(status, mem->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
    MASW_CUDA_TRY(cudaMemsetAsync(mem->d_status, 0, sizeof(int), st));
  }
  MASW_CUDA_TRY(cudaStreamSynchronize(st));
  return MASW_OK;
}

extern "C" int mem_update(masw_mem* mem, int layer, const void* k_raw, const void* v_raw, int n_raw, const void* h_g,
                          const void* Wk_g, const void* Wv_g, const int32_t* slot_pos, const uint8_t* active,
                          void* stream) {
  MASW_REQUIRE(mem != nullptr, MASW_EINVAL, "mem_update: null handle");
  { const int rc = flush_counters(mem, static_cast<cudaStream_t>(stream)); if (rc != MASW_OK) return rc; }
  mem->kv_clean = false;   // this call writes the counters or the arena: the next attention launch reads them behind its wait
  MASW_REQUIRE(layer >= 0 && layer < mem->cfg.n_layers, MASW_EINVAL, "mem_update: layer %d out of range", layer);
  const masw_config& c = mem->cfg;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const bool has_raw = (k_raw != nullptr || v_raw != nullptr);
  const bool has_slot = (h_g != nullptr || Wk_g != nullptr || Wv_g != nullptr);
  if (has_raw) {
    MASW_REQUIRE(k_raw != nullptr && v_raw != nullptr, MASW_EINVAL, "mem_update: k_raw and v_raw must both be given");
    MASW_REQUIRE(n_raw >= 1 && n_raw <= c.gamma_max, MASW_EINVAL, "mem_update: n_raw %d outside [1, gamma_max = %d]", n_raw, c.gamma_max);
    MASW_REQUIRE(aligned16(k_raw) && aligned16(v_raw), MASW_EALIGN, "mem_update: raw KV pointers must be 16-byte aligned");
  }
  if (has_slot) {
    MASW_REQUIRE(h_g != nullptr && Wk_g != nullptr && Wv_g != nullptr && slot_pos != nullptr, MASW_EINVAL,
                 "mem_update: h_g, Wk_g, Wv_g and slot_pos must all be given for a slot");
    MASW_REQUIRE(aligned16(h_g) && aligned16(Wk_g) && aligned16(Wv_g), MASW_EALIGN,
                 "mem_update: slot inputs must be 16-byte aligned");
    MASW_REQUIRE(mem->slots_upper < c.max_slots, MASW_ECAPACITY, "mem_update: slot region full (%d slots)", c.max_slots);
  }
  if (has_raw) {
    dim3 grid(n_raw, c.n_kv_heads, c.batch);
    append_raw_kernel<<<grid, c.head_dim / 8, 0, st>>>(mem->k_layer(layer), mem->v_layer(layer),
                                                       static_cast<const __nv_bfloat16*>(k_raw),
                                                       static_cast<const __nv_bfloat16*>(v_raw), mem->d_t, geom_of(mem), n_raw);
    count_launch();
    MASW_CUDA_TRY(cudaGetLastError());
  }
  if (has_slot) {
    dim3 grid(kProjKSplit, c.n_kv_heads, 2);
    if (c.head_dim == 64) {
      slot_project_kernel<64><<<grid, kProjThreads, 0, st>>>(
          mem->k_layer(layer), mem->v_layer(layer), static_cast<const __nv_bfloat16*>(h_g),
          static_cast<const __nv_bfloat16*>(Wk_g), static_cast<const __nv_bfloat16*>(Wv_g), slot_pos, active, mem->d_slots,
          mem->d_proj_part, mem->d_tickets_proj, mem->d_status, geom_of(mem), c.d_model, mem->rope_base);
    } else {
      slot_project_kernel<128><<<grid, kProjThreads, 0, st>>>(
          mem->k_layer(layer), mem->v_layer(layer), static_cast<const __nv_bfloat16*>(h_g),
          static_cast<const __nv_bfloat16*>(Wk_g), static_cast<const __nv_bfloat16*>(Wv_g), slot_pos, active, mem->d_slots,
          mem->d_proj_part, mem->d_tickets_proj, mem->d_status, geom_of(mem), c.d_model, mem->rope_base);
    }
    count_launch();
    MASW_CUDA_TRY(cudaGetLastError());
  }
  return MASW_OK;
}

extern "C" int mem_advance(masw_mem* mem, int n_tokens, int add_slot, const uint8_t* active, void* stream) {
  MASW_REQUIRE(mem != nullptr, MASW_EINVAL, "mem_advance: null handle");
  MASW_REQUIRE(n_tokens >= 0 && n_tokens <= mem->cfg.gamma_max, MASW_EINVAL, "mem_advance: n_tokens %d outside [0, gamma_max]", n_tokens);
  { const int rc = flush_counters(mem, static_cast<cudaStream_t>(stream)); if (rc != MASW_OK) return rc; }
  mem->kv_clean = false;   // this call writes the counters or the arena: the next attention launch reads them behind its wait
  if (add_slot) {
    MASW_REQUIRE(mem->slots_upper < mem->cfg.max_slots, MASW_ECAPACITY, "mem_advance: slot region full");
    mem->slots_upper += 1;
  }
  return launch_advance(mem, n_tokens, add_slot ? 1 : 0, active, static_cast<cudaStream_t>(stream));
}

extern "C" int mem_advance_deferred(masw_mem* mem, int n_tokens, int add_slot) {
  MASW_REQUIRE(mem != nullptr, MASW_EINVAL, "mem_advance_deferred: null handle");
  MASW_REQUIRE(n_tokens >= 0 && n_tokens <= mem->cfg.gamma_max, MASW_EINVAL, "mem_advance_deferred: n_tokens %d outside [0, gamma_max]",
               n_tokens);
  if (add_slot) {
    MASW_REQUIRE(mem->slots_upper < mem->cfg.max_slots, MASW_ECAPACITY, "mem_advance_deferred: slot region full");
    mem->slots_upper += 1;
    mem->pend_m += 1;
  }
  mem->pend_t += n_tokens;   // nothing is launched and nothing on the device changes: kv_clean stays as it is
  return MASW_OK;
}

extern "C" int mem_flush(masw_mem* mem, void* stream) {
  MASW_REQUIRE(mem != nullptr, MASW_EINVAL, "mem_flush: null handle");
  return flush_counters(mem, static_cast<cudaStream_t>(stream));
}

extern "C" int mem_rollback(masw_mem* mem, const int32_t* t_keep, const int32_t* slots_keep, int slots_keep_max,
                            void* stream) {
  MASW_REQUIRE(mem != nullptr && t_keep != nullptr && slots_keep != nullptr, MASW_EINVAL, "mem_rollback: null argument");
  mem->kv_clean = false;   // this call writes the counters or the arena: the next attention launch reads them behind its wait
  if (slots_keep_max >= 0) mem->slots_upper = std::min(mem->slots_upper, slots_keep_max);
  const int B = mem->cfg.batch;
  {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((B + 127) / 128, 1, 1);
    cfg.blockDim = dim3(128, 1, 1);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = counters_overlap(mem);
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    MASW_CUDA_TRY(cudaLaunchKernelEx(&cfg, rollback_kernel, mem->d_t, mem->d_slots, t_keep, slots_keep, B, mem->pend_t, mem->pend_m,
                                     mem->cfg.max_slots));
  }
  mem->pend_t = 0;   // a deferred counter update was applied by this launch
  mem->pend_m = 0;
  count_launch();
  return MASW_OK;
}
