// accept_reject: the standard speculative-sampling accept/reject rule, greedy and sampled, as one
// kernel launch.  Sampling uses 40-bit fixed-point integer weights built from a fixed recipe of IEEE
// double operations, so every decision is exact integer arithmetic and reproducible bit for bit.
#include <mutex>

#include "common.cuh"

namespace masw {

constexpr int kAcceptThreads = 512;
constexpr int kFracBits = 40;

struct RowInfo {
  double zmax_p, zmax_q;
  unsigned long long Zp, Zq;
  int argmax_p;
  int accept;
};

struct AcceptWs {
  size_t off_tickets, off_rows, total;
};

static inline AcceptWs accept_ws(int B, int gamma) {
  AcceptWs w;
  size_t off = 0;
  w.off_tickets = off; off += (sizeof(int) * B + 255) / 256 * 256;
  w.off_rows = off;    off += (sizeof(RowInfo) * B * (gamma + 1) + 255) / 256 * 256;
  w.total = off;
  return w;
}

__device__ __forceinline__ float bf16_bits_to_float(unsigned short bits) {
  return __uint_as_float(static_cast<unsigned int>(bits) << 16);
}

// exp(e) for e <= 0 from IEEE double multiply / add / rint / exact scaling only (never fused):
// n = rint(e * log2 e); r = (e - n * LN2_HI) - n * LN2_LO; degree-13 Taylor polynomial in Horner form.
__device__ __forceinline__ double spec_exp(double e) {
  if (e < -64.0) return 0.0;
  const double kInvFact[14] = {1.0 / 1.0, 1.0 / 1.0, 1.0 / 2.0, 1.0 / 6.0, 1.0 / 24.0, 1.0 / 120.0, 1.0 / 720.0,
                               1.0 / 5040.0, 1.0 / 40320.0, 1.0 / 362880.0, 1.0 / 3628800.0, 1.0 / 39916800.0,
                               1.0 / 479001600.0, 1.0 / 6227020800.0};
  const double n = rint(__dmul_rn(e, 1.4426950408889634));
  const double r = __dsub_rn(__dsub_rn(e, __dmul_rn(n, 6.93147180369123816490e-01)),
                             __dmul_rn(n, 1.90821492927058770002e-10));
  double p = kInvFact[13];
#pragma unroll
  for (int k = 12; k >= 0; --k) p = __dadd_rn(__dmul_rn(p, r), kInvFact[k]);
  return scalbn(p, static_cast<int>(n));
}

__device__ __forceinline__ unsigned long long int_weight(float x, double temp, double zmax) {
  const double z = __ddiv_rn(static_cast<double>(x), temp);
  const double w = spec_exp(__dsub_rn(z, zmax));
  return __double2ull_rd(scalbn(w, kFracBits));
}

struct MaxIdx {
  float v;
  int i;
};
__device__ __forceinline__ MaxIdx better(MaxIdx a, MaxIdx b) {
  // larger value wins; equal values: lower index wins
  if (b.v > a.v || (b.v == a.v && b.i < a.i)) return b;
  return a;
}

__device__ MaxIdx block_argmax(MaxIdx mine, MaxIdx* sh) {
  for (int o = 16; o > 0; o >>= 1) {
    MaxIdx other;
    other.v = __shfl_xor_sync(0xffffffffu, mine.v, o);
    other.i = __shfl_xor_sync(0xffffffffu, mine.i, o);
    mine = better(mine, other);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();
  if (lane == 0) sh[warp] = mine;
  __syncthreads();
  MaxIdx r = sh[0];
  for (int w = 1; w < kAcceptThreads / 32; ++w) r = better(r, sh[w]);
  return r;
}

__device__ unsigned long long block_sum_u64(unsigned long long mine, unsigned long long* sh) {
  for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();
  if (lane == 0) sh[warp] = mine;
  __syncthreads();
  unsigned long long r = 0;
  for (int w = 0; w < kAcceptThreads / 32; ++w) r += sh[w];
  return r;
}

// Draws the smallest j whose inclusive prefix sum of weights exceeds (U * total) >> 24.  Each thread
// owns a contiguous chunk of the row; weight(j) is recomputed when the owning thread rescans.
// Returns -1 when the total is zero.  All threads get the result.
template <typename WeightFn>
__device__ int block_draw(int V, unsigned int U, WeightFn weight, unsigned long long* sh_u64, int* sh_int) {
  const int chunk = (V + kAcceptThreads - 1) / kAcceptThreads;
  const int j0 = min(V, static_cast<int>(threadIdx.x) * chunk), j1 = min(V, j0 + chunk);
  unsigned long long local = 0;
  for (int j = j0; j < j1; ++j) local += weight(j);
  __syncthreads();
  sh_u64[threadIdx.x] = local;
  if (threadIdx.x == 0) *sh_int = -1;
  __syncthreads();
  // exclusive offset of this thread's chunk and the row total (serial over 512 values: negligible)
  unsigned long long offset = 0, total = 0;
  for (int i = 0; i < kAcceptThreads; ++i) {
    const unsigned long long v = sh_u64[i];
    if (i < static_cast<int>(threadIdx.x)) offset += v;
    total += v;
  }
  if (total != 0) {
    const unsigned long long tau =
        static_cast<unsigned long long>((static_cast<unsigned __int128>(U) * total) >> 24);
    if (tau >= offset && tau < offset + local) {
      unsigned long long run = offset;
      for (int j = j0; j < j1; ++j) {
        run += weight(j);
        if (run > tau) { *sh_int = j; break; }
      }
    }
  }
  __syncthreads();
  const int r = *sh_int;
  __syncthreads();
  return r;
}

// grid (gamma + 1, B), kAcceptThreads threads.  Block (i, b) scores target row i (and draft row i);
// the last block of sequence b to finish (atomic ticket) walks the rows and makes the final draw.
__global__ void __launch_bounds__(kAcceptThreads)
accept_reject_kernel(const unsigned short* tl, const unsigned short* dl, const int* draft_tokens, const float* uniforms,
                     int gamma, int V, float temperature, int* n_accepted, int* out_tokens, int* status,
                     int* tickets, RowInfo* rows) {
  __shared__ MaxIdx sh_mi[kAcceptThreads / 32];
  __shared__ unsigned long long sh_u64[kAcceptThreads];
  __shared__ int sh_int;
  __shared__ int sh_last;

  // launched with programmatic stream serialisation (accept_reject): the blocks may be set up while the kernel in
  // front still runs; nothing is read before it has completed, and the successor may be set up at once
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const int i = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x;
  const bool sampling = temperature > 0.f;
  const double temp = static_cast<double>(temperature);
  const unsigned short* prow = tl + (static_cast<size_t>(b) * (gamma + 1) + i) * V;
  const unsigned short* qrow = (sampling && i < gamma) ? dl + (static_cast<size_t>(b) * gamma + i) * V : nullptr;
  RowInfo* info = rows + static_cast<size_t>(b) * (gamma + 1) + i;

  // ---- pass 1: arg-max of the target row (lowest index on ties), max of the draft row
  MaxIdx mp{-INFINITY, 0x7fffffff}, mq{-INFINITY, 0x7fffffff};
  bool bad = false;
  // rows that start on a 16-byte boundary (V a multiple of 8, aligned base) are read eight logits per load,
  // with all of a thread's loads in flight together: the pass is a latency chain otherwise
  const bool vec = (V % 8 == 0) && ((reinterpret_cast<uintptr_t>(tl) | reinterpret_cast<uintptr_t>(dl)) % 16 == 0);
  auto scan_row = [&](const unsigned short* row, MaxIdx& m) {
    if (vec) {
      const uint4* row4 = reinterpret_cast<const uint4*>(row);
      const int n4 = V / 8;
      constexpr int kInFlight = 8;   // 16-byte loads per thread and round trip (a 128K-entry row takes four trips)
      for (int j0 = tid; j0 < n4; j0 += kAcceptThreads * kInFlight) {
        uint4 w[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
          const int j4 = j0 + u * kAcceptThreads;
          w[u] = j4 < n4 ? __ldg(row4 + j4) : make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);   // -inf pads
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
          const int j4 = j0 + u * kAcceptThreads;
          if (j4 >= n4) continue;
          const unsigned int word[4] = {w[u].x, w[u].y, w[u].z, w[u].w};
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const float x = bf16_bits_to_float(static_cast<unsigned short>(word[k >> 1] >> (16 * (k & 1))));
            bad |= !(fabsf(x) <= 3.0e38f);
            m = better(m, MaxIdx{x, j4 * 8 + k});
          }
        }
      }
    } else {
      for (int j = tid; j < V; j += kAcceptThreads) {
        const float x = bf16_bits_to_float(__ldg(row + j));
        bad |= !(fabsf(x) <= 3.0e38f);
        m = better(m, MaxIdx{x, j});
      }
    }
  };
  scan_row(prow, mp);
  if (qrow) scan_row(qrow, mq);
  mp = block_argmax(mp, sh_mi);
  if (qrow) mq = block_argmax(mq, sh_mi);
  if (bad && status) atomicOr(status, MASW_STATUS_BAD_LOGIT);

  int accept = 0;
  unsigned long long Zp = 0, Zq = 0;
  double zmax_p = 0.0, zmax_q = 0.0;
  if (!sampling) {
    if (i < gamma) {
      const int x = draft_tokens[b * gamma + i];
      if ((x < 0 || x >= V) && tid == 0 && status) atomicOr(status, MASW_STATUS_BAD_TOKEN);
      accept = (x == mp.i) ? 1 : 0;
    }
  } else {
    // ---- pass 2: integer weights, their sums, and the accept test of this row
    zmax_p = __ddiv_rn(static_cast<double>(mp.v), temp);
    unsigned long long sp = 0, sq = 0;
    for (int j = tid; j < V; j += kAcceptThreads) sp += int_weight(bf16_bits_to_float(__ldg(prow + j)), temp, zmax_p);
    Zp = block_sum_u64(sp, sh_u64);
    if (qrow) {
      zmax_q = __ddiv_rn(static_cast<double>(mq.v), temp);
      for (int j = tid; j < V; j += kAcceptThreads) sq += int_weight(bf16_bits_to_float(__ldg(qrow + j)), temp, zmax_q);
      Zq = block_sum_u64(sq, sh_u64);
      int x = draft_tokens[b * gamma + i];
      if (x < 0 || x >= V) {
        if (tid == 0 && status) atomicOr(status, MASW_STATUS_BAD_TOKEN);
        x = min(max(x, 0), V - 1);
      }
      const unsigned long long Ipx = int_weight(bf16_bits_to_float(__ldg(prow + x)), temp, zmax_p);
      const unsigned long long Iqx = int_weight(bf16_bits_to_float(__ldg(qrow + x)), temp, zmax_q);
      const unsigned int U = static_cast<unsigned int>(floorf(uniforms[b * (gamma + 1) + i] * 16777216.0f));
      const unsigned __int128 lhs = static_cast<unsigned __int128>(U) * Iqx * Zp;
      const unsigned __int128 rhs = (static_cast<unsigned __int128>(Ipx) << 24) * Zq;
      accept = (lhs < rhs) ? 1 : 0;
    }
  }
  if (tid == 0) {
    info->zmax_p = zmax_p; info->zmax_q = zmax_q;
    info->Zp = Zp; info->Zq = Zq;
    info->argmax_p = mp.i; info->accept = accept;
  }

  // ---- ticket: the last block of this sequence finishes the job
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int ticket = atomicAdd(&tickets[b], 1);
    sh_last = (ticket == gamma) ? 1 : 0;
  }
  __syncthreads();
  if (sh_last == 0) return;
  __threadfence();

  const volatile RowInfo* seq = rows + static_cast<size_t>(b) * (gamma + 1);
  int n = 0;
  while (n < gamma && seq[n].accept != 0) ++n;
  int final_tok;
  if (!sampling) {
    final_tok = seq[n].argmax_p;
  } else {
    const unsigned int U = static_cast<unsigned int>(floorf(uniforms[b * (gamma + 1) + gamma] * 16777216.0f));
    const unsigned short* pr = tl + (static_cast<size_t>(b) * (gamma + 1) + n) * V;
    const double zp = seq[n].zmax_p;
    if (n < gamma) {
      const unsigned short* qr = dl + (static_cast<size_t>(b) * gamma + n) * V;
      const double zq = seq[n].zmax_q;
      const unsigned long long Zpn = seq[n].Zp, Zqn = seq[n].Zq;
      auto resid = [&](int j) -> unsigned long long {
        const unsigned __int128 a = static_cast<unsigned __int128>(int_weight(bf16_bits_to_float(__ldg(pr + j)), temp, zp)) * Zqn;
        const unsigned __int128 c = static_cast<unsigned __int128>(int_weight(bf16_bits_to_float(__ldg(qr + j)), temp, zq)) * Zpn;
        return a > c ? static_cast<unsigned long long>((a - c) >> 48) : 0ull;
      };
      final_tok = block_draw(V, U, resid, sh_u64, &sh_int);
      if (final_tok < 0) final_tok = seq[n].argmax_p;
    } else {
      auto wp = [&](int j) -> unsigned long long { return int_weight(bf16_bits_to_float(__ldg(pr + j)), temp, zp); };
      final_tok = block_draw(V, U, wp, sh_u64, &sh_int);
      if (final_tok < 0) final_tok = seq[n].argmax_p;
    }
  }
  if (tid == 0) n_accepted[b] = n;
  for (int k = tid; k <= gamma; k += kAcceptThreads) {
    int tok = -1;
    if (k < n) tok = draft_tokens[b * gamma + k];
    else if (k == n) tok = final_tok;
    out_tokens[b * (gamma + 1) + k] = tok;
  }
  if (tid == 0) tickets[b] = 0;
}

}  // namespace masw

namespace masw {
// Sampling keeps the sum of the residual weights in 64 bits.  Its largest value, reached when p and q are flat
// on disjoint halves of the vocabulary, is (V / 2)^2 2^32 = V^2 2^30, which fits while V < 2^17.
constexpr int kMaxSamplingVocab = 131071;
}  // namespace masw

using namespace masw;

extern "C" size_t accept_workspace_bytes(int batch, int gamma, int vocab) {
  if (batch < 1 || gamma < 1 || vocab < 1) return 0;
  return accept_ws(batch, gamma).total;
}

extern "C" int accept_reject(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                             const float* uniforms, int batch, int gamma, int vocab, float temperature,
                             int32_t* n_accepted, int32_t* out_tokens, int32_t* status, void* workspace,
                             size_t workspace_bytes, void* stream) {
  MASW_REQUIRE(target_logits != nullptr && draft_tokens != nullptr && n_accepted != nullptr && out_tokens != nullptr &&
                   workspace != nullptr,
               MASW_EINVAL, "accept_reject: null argument");
  MASW_REQUIRE(batch >= 1 && gamma >= 1 && gamma <= 64 && vocab >= 1, MASW_EINVAL, "accept_reject: bad batch/gamma/vocab");
  MASW_REQUIRE(temperature >= 0.f && temperature == temperature, MASW_EINVAL, "accept_reject: temperature must be >= 0");
  if (temperature > 0.f) {
    MASW_REQUIRE(draft_logits != nullptr && uniforms != nullptr, MASW_EINVAL,
                 "accept_reject: sampling needs draft_logits and uniforms");
    MASW_REQUIRE(vocab <= kMaxSamplingVocab, MASW_EINVAL,
                 "accept_reject: sampling keeps 64-bit weight sums, exact only for vocab <= %d (got %d)", kMaxSamplingVocab, vocab);
  }
  MASW_REQUIRE((reinterpret_cast<uintptr_t>(workspace) & 15) == 0, MASW_EALIGN, "accept_reject: workspace must be 16-byte aligned");
  const AcceptWs w = accept_ws(batch, gamma);
  MASW_REQUIRE(workspace_bytes >= w.total, MASW_ECAPACITY, "accept_reject: workspace %zu < %zu bytes", workspace_bytes, w.total);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(gamma + 1, batch, 1);
    cfg.blockDim = dim3(kAcceptThreads, 1, 1);
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    MASW_CUDA_TRY(cudaLaunchKernelEx(&cfg, accept_reject_kernel, static_cast<const unsigned short*>(target_logits),
                                     static_cast<const unsigned short*>(draft_logits), draft_tokens, uniforms, gamma, vocab,
                                     temperature, n_accepted, out_tokens, status, reinterpret_cast<int*>(ws + w.off_tickets),
                                     reinterpret_cast<RowInfo*>(ws + w.off_rows)));
  }
  count_launch();
  return MASW_OK;
}

// ---------------------------------------------------------------------------------------------------
// accept_reject_static: the same kernel with its scratch in a fixed device array owned by the library.
namespace masw {

constexpr int kStaticMaxBatch = 64;
constexpr int kStaticMaxGamma = 16;
constexpr size_t kStaticTicketBytes = 256;   // int tickets[kStaticMaxBatch]
constexpr size_t kStaticScratchBytes = kStaticTicketBytes + sizeof(RowInfo) * kStaticMaxBatch * (kStaticMaxGamma + 1);

// Lives in every device that loads the library, from load until the process exits (about 43 KB).
// In host code this name is only a handle for the runtime, never a device address: the address is
// looked up per device with cudaGetSymbolAddress below and that pointer is what the kernel receives.
static __device__ __align__(256) unsigned char g_accept_scratch[kStaticScratchBytes];

static std::mutex g_static_mu;
static unsigned char* g_static_ptr[kMaxDevices] = {};

// Device address of g_accept_scratch on the current device; resolved once per device.
static int static_scratch(unsigned char** out) {
  int dev = -1;
  MASW_CUDA_TRY(cudaGetDevice(&dev));
  MASW_REQUIRE(dev >= 0 && dev < kMaxDevices, MASW_EINVAL, "accept_reject_static: device index %d not supported", dev);
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (g_static_ptr[dev] == nullptr) {
    void* ptr = nullptr;
    MASW_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_accept_scratch));
    MASW_REQUIRE(ptr != nullptr, MASW_ECUDA, "accept_reject_static: no device address for the scratch array");
    g_static_ptr[dev] = static_cast<unsigned char*>(ptr);
  }
  *out = g_static_ptr[dev];
  return MASW_OK;
}

}  // namespace masw

extern "C" int accept_reject_static(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                                    const float* uniforms, int batch, int gamma, int vocab, float temperature,
                                    int32_t* n_accepted, int32_t* out_tokens, int32_t* status, void* stream) {
  MASW_REQUIRE(target_logits != nullptr && draft_tokens != nullptr && n_accepted != nullptr && out_tokens != nullptr,
               MASW_EINVAL, "accept_reject_static: null argument");
  MASW_REQUIRE(batch >= 1 && gamma >= 1 && vocab >= 1, MASW_EINVAL, "accept_reject_static: bad batch/gamma/vocab");
  MASW_REQUIRE(batch <= kStaticMaxBatch && gamma <= kStaticMaxGamma, MASW_ECAPACITY,
               "accept_reject_static: batch %d / gamma %d exceed the built-in scratch (batch <= %d, gamma <= %d); "
               "use accept_reject with a caller-provided workspace",
               batch, gamma, kStaticMaxBatch, kStaticMaxGamma);
  MASW_REQUIRE(temperature >= 0.f && temperature == temperature, MASW_EINVAL, "accept_reject_static: temperature must be >= 0");
  if (temperature > 0.f) {
    MASW_REQUIRE(draft_logits != nullptr && uniforms != nullptr, MASW_EINVAL,
                 "accept_reject_static: sampling needs draft_logits and uniforms");
    MASW_REQUIRE(vocab <= kMaxSamplingVocab, MASW_EINVAL,
                 "accept_reject_static: sampling keeps 64-bit weight sums, exact only for vocab <= %d (got %d)", kMaxSamplingVocab, vocab);
  }
  unsigned char* scratch = nullptr;
  int rc = static_scratch(&scratch);
  if (rc != MASW_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the previous call left: the tickets must start at zero
  MASW_CUDA_TRY(cudaMemsetAsync(scratch, 0, kStaticTicketBytes, st));
  dim3 grid(gamma + 1, batch);
  accept_reject_kernel<<<grid, kAcceptThreads, 0, st>>>(
      static_cast<const unsigned short*>(target_logits), static_cast<const unsigned short*>(draft_logits), draft_tokens,
      uniforms, gamma, vocab, temperature, n_accepted, out_tokens, status, reinterpret_cast<int*>(scratch),
      reinterpret_cast<RowInfo*>(scratch + kStaticTicketBytes));
  count_launch();
  MASW_CUDA_TRY(cudaGetLastError());
  return MASW_OK;
}
