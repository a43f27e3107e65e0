// Shared host/device helpers of the MASW library (sm_100a only).
#pragma once

#include <atomic>

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>

#include "../../include/masw.h"

namespace masw {

// ------------------------------------------------------------------------------------------------
// host-side error plumbing
void set_error(const char* fmt, ...);
void count_launch(int n = 1);
int check_cuda(cudaError_t e, const char* what);
constexpr int kMaxDevices = 64;   // per-device caches (kernel attributes, SM counts, symbol addresses) are arrays of this size
int current_device();             // index of the current CUDA device, clamped to [0, kMaxDevices)
int sm_count();                   // SM count of the current device

#define MASW_CUDA_TRY(expr)                                        \
  do {                                                             \
    int _rc = ::masw::check_cuda((expr), #expr);                   \
    if (_rc != MASW_OK) return _rc;                                \
  } while (0)

#define MASW_REQUIRE(cond, code, ...)                              \
  do {                                                             \
    if (!(cond)) {                                                 \
      ::masw::set_error(__VA_ARGS__);                              \
      return (code);                                               \
    }                                                              \
  } while (0)

// Raises a kernel's dynamic shared-memory limit once per device (the attribute is per device, and a
// process may drive several).  `once` is a static object of the launching function.
struct PerDeviceOnce { std::atomic<bool> done[kMaxDevices]; };
template <typename Kern>
static inline int set_smem_once(Kern kern, int bytes, PerDeviceOnce& once) {
  const int dev = current_device();
  if (!once.done[dev].load(std::memory_order_acquire)) {
    MASW_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes));
    once.done[dev].store(true, std::memory_order_release);
  }
  return MASW_OK;
}

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Encodes a 4-D bf16 tensor map (head_dim, entries, kv heads, batch) with a [64 x box_rows] box and
// 128-byte swizzle.  Strides are in elements.
int encode_kv_tensor_map(CUtensorMap* out, const void* base, int head_dim, int64_t entries, int n_kv_heads,
                         int batch, int64_t stride_n, int64_t stride_h, int64_t stride_b, int box_rows);

// Tensor maps (K and V) of a caller-described cache with a [64 x box_rows] box, from a small cache keyed by
// the description (encoding costs a few microseconds of host time).
int get_kv_maps(const masw_kv_desc& kv, int box_rows, CUtensorMap* tk, CUtensorMap* tv);

// Tensor map of a pool of FP8 pages ([page][kv head][128][128] bytes), box = one page of one head.
int encode_fp8_page_map(CUtensorMap* out, const void* base, int n_kv_heads, int n_pages);

// ------------------------------------------------------------------------------------------------
// device-side primitives
#ifdef __CUDACC__

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}

__device__ __forceinline__ void fence_mbar_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

__device__ __forceinline__ void fence_proxy_async() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// One poll that lets the hardware park the thread until the phase completes or `ns` nanoseconds have passed:
// a waiting warp then issues a handful of instructions per wait instead of spinning in the issue slots that
// the working warps of the same scheduler need.
__device__ __forceinline__ bool mbar_try_wait_parked(uint64_t* bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(ns)
      : "memory");
  return ok != 0;
}

// Bounded wait: gives up after `limit` polls (kWaitLimit unless the launch says otherwise), so a lost copy
// can never hang the GPU.  Returns false on give-up.  The first poll returns at once (short waits stay
// cheap), later ones park the thread for up to kParkNs each, which bounds the whole wait to a few seconds.
constexpr int kWaitLimit = 1 << 20;
constexpr uint32_t kParkNs = 4000;
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, int limit = kWaitLimit) {
  if (mbar_try_wait(bar, parity)) return true;
  for (int i = 0; i < limit; ++i) {
    if (mbar_try_wait_parked(bar, parity, kParkNs)) return true;
  }
  return false;
}

// One 4-D tiled bulk copy global -> shared; completion is signalled on `bar` (transaction bytes).
__device__ __forceinline__ void tma_load_4d(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int c0, int c1,
                                            int c2, int c3, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4, %5, %6}], [%2], %7;"
      ::"r"(smem_u32(smem_dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1),
      "r"(c2), "r"(c3), "l"(policy)
      : "memory");
}

// Prefetch of one box into L2 only (no shared-memory destination, no completion to wait for).
__device__ __forceinline__ void tma_prefetch_4d(const CUtensorMap* map, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.prefetch.tensor.4d.L2.global.tile [%0, {%1, %2, %3, %4}];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
}

__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}

__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                                  uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x2(uint32_t& r0, uint32_t& r1, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}

__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t& r0, uint32_t& r1, uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0,%1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}

// A hint that brings one line into L2; no value is read, so it may name memory another kernel is still writing.
__device__ __forceinline__ void prefetch_l2(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

// D += A(16x16, row) * B(16x8, col), bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// The limit of the kernels' bounded waits: a launch parameter in the developer build (a test shortens it to make a
// wait run out), the compile-time constant in the product build (the polling loops compile tighter with it).
#ifdef MASW_TRACE
#define MASW_WAIT_LIMIT(p) ((p).wait_limit)
#else
#define MASW_WAIT_LIMIT(p) (::masw::kWaitLimit)
#endif

constexpr int kTraceWords = 32;   // developer build: 64-bit words of one CTA's stamp record

// Phase stamps of the developer build (-DMASW_TRACE): thread `who` of the CTA writes %globaltimer into word
// `slot` of the CTA's record.  The product build compiles them out.
#ifdef MASW_TRACE
#define MASW_STAMP_BY(tr, who, slot)                                              \
  do {                                                                            \
    if ((tr) != nullptr && threadIdx.x == (who)) {                                \
      long long t_;                                                               \
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_) : : "memory");         \
      (tr)[slot] = t_;                                                            \
    }                                                                             \
  } while (0)
#else
#define MASW_STAMP_BY(tr, who, slot) do { } while (0)
#endif
#define MASW_STAMP(tr, slot) MASW_STAMP_BY(tr, 0, slot)
// The SM's cycle counter instead (cheap to read, comparable only inside one CTA): thread 0 of the CTA.
#ifdef MASW_TRACE
#define MASW_CLOCK(tr, slot)                                                      \
  do {                                                                            \
    if ((tr) != nullptr && threadIdx.x == 0) (tr)[slot] = clock64();              \
  } while (0)
#else
#define MASW_CLOCK(tr, slot) do { } while (0)
#endif

#endif  // __CUDACC__

}  // namespace masw
