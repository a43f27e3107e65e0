// Host-side plumbing shared by all entry points: error text, launch accounting, device queries and
// TMA descriptor encoding (through the driver entry point, so the library links without libcuda).
#include <atomic>
#include <cstdarg>
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace masw {

static thread_local char g_error[512] = "";
static std::atomic<uint64_t> g_launches{0};

void set_error(const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_error, sizeof(g_error), fmt, ap);
  va_end(ap);
}

void count_launch(int n) { g_launches.fetch_add(static_cast<uint64_t>(n), std::memory_order_relaxed); }

int check_cuda(cudaError_t e, const char* what) {
  if (e == cudaSuccess) return MASW_OK;
  set_error("CUDA error %d (%s) in %s", static_cast<int>(e), cudaGetErrorString(e), what);
  return MASW_ECUDA;
}

int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
  return dev;
}

// SM count of the current device, cached per device (a process may drive several GPUs)
int sm_count() {
  static std::atomic<int> cached[kMaxDevices];
  const int dev = current_device();
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
  cached[dev].store(n, std::memory_order_relaxed);
  return n;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess) {
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
  });
  return fn;
}

int encode_kv_tensor_map(CUtensorMap* out, const void* base, int head_dim, int64_t entries, int n_kv_heads,
                         int batch, int64_t stride_n, int64_t stride_h, int64_t stride_b, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  MASW_REQUIRE(fn != nullptr, MASW_ECUDA, "cuTensorMapEncodeTiled is unavailable (no CUDA driver?)");
  cuuint64_t dims[4] = {static_cast<cuuint64_t>(head_dim), static_cast<cuuint64_t>(entries),
                        static_cast<cuuint64_t>(n_kv_heads), static_cast<cuuint64_t>(batch)};
  cuuint64_t strides[3] = {static_cast<cuuint64_t>(stride_n) * 2, static_cast<cuuint64_t>(stride_h) * 2,
                           static_cast<cuuint64_t>(stride_b) * 2};
  // a degenerate dimension may carry any stride; keep the encoder's stride checks satisfied
  if (n_kv_heads == 1 && strides[1] < strides[0] * dims[1]) strides[1] = strides[0] * dims[1];
  if (batch == 1 && strides[2] < strides[1] * dims[2]) strides[2] = strides[1] * dims[2];
  cuuint32_t box[4] = {64u, static_cast<cuuint32_t>(box_rows), 1u, 1u};
  cuuint32_t elem[4] = {1u, 1u, 1u, 1u};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  MASW_REQUIRE(r == CUDA_SUCCESS, MASW_ECUDA, "cuTensorMapEncodeTiled failed with %d", static_cast<int>(r));
  return MASW_OK;
}

// A pool of FP8 pages [page][kv head][128 entries][128 bytes] as a 4-D byte tensor (byte of the entry, entry of
// the page, kv head, page) with a [128 x 128] box and 128-byte swizzle.
int encode_fp8_page_map(CUtensorMap* out, const void* base, int n_kv_heads, int n_pages) {
  EncodeTiledFn fn = encode_fn();
  MASW_REQUIRE(fn != nullptr, MASW_ECUDA, "cuTensorMapEncodeTiled is unavailable (no CUDA driver?)");
  cuuint64_t dims[4] = {128u, 128u, static_cast<cuuint64_t>(n_kv_heads), static_cast<cuuint64_t>(n_pages)};
  cuuint64_t strides[3] = {128u, 128u * 128u, static_cast<cuuint64_t>(n_kv_heads) * 128u * 128u};
  cuuint32_t box[4] = {128u, 128u, 1u, 1u};
  cuuint32_t elem[4] = {1u, 1u, 1u, 1u};
  CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4, const_cast<void*>(base), dims, strides, box, elem,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  MASW_REQUIRE(r == CUDA_SUCCESS, MASW_ECUDA, "cuTensorMapEncodeTiled (FP8 pages) failed with %d", static_cast<int>(r));
  return MASW_OK;
}

}  // namespace masw

extern "C" {

const char* masw_last_error(void) { return masw::g_error; }

uint64_t masw_launch_count(void) { return masw::g_launches.load(std::memory_order_relaxed); }

const char* masw_version(void) { return "masw-b200 0.1 (sm_100a)"; }

}  // extern "C"
