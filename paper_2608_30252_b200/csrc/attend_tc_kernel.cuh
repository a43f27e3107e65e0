// tcgen05 / TMEM variant of the split-K attention kernel for head_dim 128 (verify_attend).
//
// The decode-style query tile has few rows (tokens x group heads <= 64) but each KV tile has many
// entries, so the tensor-core M dimension is given to the ENTRIES and the small row count becomes N:
//
//   MMA1:  S^T[128 entries x NQ rows] = K[128 x 128 dims] . Q^T        (A = K tile, B = Q tile, both K-major)
//   MMA2:  O^T[128 dims x NQ rows]   += V^T[128 dims x 128 entries] . P^T   (A = V tile read MN-major, B = P stored
//          [entry][row], MN-major as well: an entry's NQ probabilities are one swizzled line of 2 NQ bytes)
//
// Both accumulators live in tensor memory (TMEM); operands are read by the tensor core straight from
// the 128B-swizzled shared-memory tiles that TMA wrote, so no fragment ever passes through registers.
// Warp roles (384 threads; one CTA per SM):
//   warp 0      TMA producer (one lane): K tiles and V tiles of 128 entries into two rings (NK, NV slots);
//               it also owns the tile schedule (a static range per split plus a pool the splits of one
//               (sequence, KV head) claim from, so that a slower SM ends up with fewer tiles)
//   warp 1      MMA issuer (one lane) and owner of the TMEM allocation
//   warps 4..11 softmax, two groups of four warps, each owning half of the query rows: thread <-> TMEM lane
//               <-> entry; they read S^T with tcgen05.ld, reduce the column (= query row) maxima across the
//               128 entries with shuffles, rescale O^T in TMEM when a maximum moved, write their entry's
//               line of P as bf16 into shared memory for MMA2 (16-byte stores), keep the row sums
// S^T is double-buffered in TMEM and P in shared memory, so MMA1 of tile i+1 and P.V of tile i-1
// overlap the softmax of tile i.
// Every wait is bounded; on give-up the kernel records MASW_STATUS_WAIT_TIMEOUT and falls through.
// The split partial and the cross-split reduction are the same as in attend_kernel.
#pragma once

#include <cstddef>

#include "attend_kernel.cuh"

namespace masw {

// ---- tcgen05 primitives -------------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

// D[tmem] (+)= A[smem desc] * B[smem desc], bf16 inputs, fp32 accumulate, issued by one thread.
__device__ __forceinline__ void tc_mma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
      : "memory");
}

// Shared-memory matrix descriptors for 128B-swizzled tiles whose rows are 128 bytes apart
// (8-row groups 1024 bytes apart).  K-major: the 16-element K step stays inside one swizzle row.
// MN-major: the 64-element MN atoms are `mn_atom_bytes` apart.
__device__ __forceinline__ uint64_t tc_desc_kmajor(uint32_t saddr) {
  return static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint64_t tc_desc_mnmajor(uint32_t saddr, uint32_t mn_atom_bytes) {
  return static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(mn_atom_bytes >> 4) << 16) |
         (static_cast<uint64_t>(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// MN-major operand of 32 elements (64-byte lines, 64B swizzle: 16-byte chunk ^= (line >> 1) & 3), 8 lines per atom
__device__ __forceinline__ uint64_t tc_desc_mnmajor_sw64(uint32_t saddr) {
  return static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4) | (static_cast<uint64_t>(512 >> 4) << 16) |
         (static_cast<uint64_t>(512 >> 4) << 32) | (1ull << 46) | (4ull << 61);
}
// Instruction descriptor: fp32 accumulator, bf16 (or, with `f16`, fp16) A and B, M x N tile, operand majorness.
__host__ __device__ constexpr uint32_t tc_idesc(int M, int N, int a_mn_major, int b_mn_major, bool f16 = false) {
  return (1u << 4) | (f16 ? 0u : (1u << 7) | (1u << 10)) | (static_cast<uint32_t>(a_mn_major) << 15) |
         (static_cast<uint32_t>(b_mn_major) << 16) | (static_cast<uint32_t>(N >> 3) << 17) |
         (static_cast<uint32_t>(M >> 4) << 24);
}

// 16 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tc_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
      "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
      "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
      "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])),
      "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// two e4m3 values (the low 16 bits of `pair`) -> two fp16 values (exact: e4m3 is a subset of fp16)
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t pair) {
  uint32_t d;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(d) : "h"(static_cast<unsigned short>(pair)));
  return d;
}
__device__ __forceinline__ uint32_t hmul2_u32(uint32_t a, uint32_t b) {   // fp16x2 product, rounded to nearest
  uint32_t d;
  asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t d;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ float f16_lo_to_f32(uint32_t v) {
  float f;
  asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %1;\n\tcvt.f32.f16 %0, l;\n\t}" : "=f"(f) : "r"(v));
  return f;
}
__device__ __forceinline__ float f16_hi_to_f32(uint32_t v) {
  float f;
  asm("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %1;\n\tcvt.f32.f16 %0, h;\n\t}" : "=f"(f) : "r"(v));
  return f;
}

__device__ __forceinline__ void named_bar_sync(int id, int n_threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}

// Named barrier that also ORs a predicate over its participants: every thread learns whether any of them set it.
__device__ __forceinline__ bool named_bar_red_or(int id, int n_threads, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %3, 0;\n\t"
      "bar.red.or.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r)
      : "r"(id), "r"(n_threads), "r"(static_cast<uint32_t>(pred))
      : "memory");
  return r != 0;
}

// Butterfly over the 32 lanes of a warp for N = 32 or 16 values per lane: on return lane L holds op over
// all lanes of the original v[L % N] (N - 1 exchange shuffles, one more for N = 16).  `v` is destroyed.
template <int N, bool IS_MAX>
__device__ __forceinline__ float warp_transpose_reduce(float (&v)[N], int lane) {
  static_assert(N == 32 || N == 16, "values per lane");
#pragma unroll
  for (int off = N / 2; off >= 1; off >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int k = 0; k < off; ++k) {
      const float send = upper ? v[k] : v[k + off];
      const float keep = upper ? v[k + off] : v[k];
      const float recv = __shfl_xor_sync(0xffffffffu, send, off);
      v[k] = IS_MAX ? fmaxf(keep, recv) : keep + recv;
    }
  }
  float r = v[0];
  if (N == 16) {
    const float other = __shfl_xor_sync(0xffffffffu, r, 16);
    r = IS_MAX ? fmaxf(r, other) : r + other;
  }
  return r;
}

// FP8: the cache holds e4m3 bytes (paged, one scale per page and KV head).  Raw 16 KB tiles stream into two small
// rings; two otherwise idle warps turn each into the fp16 operand tile (same swizzled layout a bf16 tile has), and
// every MMA runs on fp16 operands (Q converted on load, P written as fp16).  NK / NV then count operand buffers.
template <int NQ, int NK, int NV, bool FP8 = false>
struct TcCfg {
  static constexpr int D = 128;
  static constexpr int kTile = 128;                    // entries per KV tile
  static constexpr int kSoftGroups = 2;                // softmax groups of four warps, each owning half of the query rows
  static constexpr int kCols = NQ / kSoftGroups;       // query rows (TMEM columns) per group
  static constexpr int kDeqWarps = 6;                  // FP8: warps 2, 3 and four more behind the softmax warps convert raw tiles
  static constexpr int kThreads = (4 + 4 * kSoftGroups + (FP8 ? 4 : 0)) * 32;
  static constexpr int kSubBytes = kTile * 128;        // one [128 x 64] bf16 box
  static constexpr int kTileBytes = 2 * kSubBytes;     // K or V tile
  static constexpr int kKRingBytes = NK * kTileBytes;   // K tiles are released as soon as S^T is computed,
  static constexpr int kVRingBytes = NV * kTileBytes;   // V tiles only after P.V: two rings of their own depth
  static constexpr int kRawTileBytes = kTile * D;      // FP8: one [128 entries x 128 bytes] box
  static constexpr int kRaw = 3;                        // FP8: raw tiles in flight per ring
  static constexpr int kRawBytes = FP8 ? 2 * kRaw * kRawTileBytes : 0;
  static constexpr int kPipeBytes = kKRingBytes + kVRingBytes + kRawBytes;
  static constexpr int kQSubBytes = NQ * 128;
  static constexpr int kQBytes = 2 * kQSubBytes;       // Q tile; the P tile has the same shape
  static constexpr int kTmemCols = (3 * NQ <= 128) ? 128 : 256;   // 2 x S^T + O^T, power of two
  static constexpr int kCtrlBytes = 1792 + 4 * NQ * 4 * 5;
  static constexpr int kSmemBytes = 1024 + kPipeBytes + 3 * kQBytes + kCtrlBytes;   // Q tile + two P tiles
  static_assert(NQ == 32 || NQ == 64, "query rows padded to 32 or 64");
  static_assert(kSmemBytes <= 232448, "shared memory budget");
};

template <int NQ>
struct TcCtrl {
  uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4], s_full[2], s_empty[2], p_full[2], p_empty[2], o_ready;
  uint64_t k8_full[4], k8_empty[4], v8_full[4], v8_empty[4];   // FP8: the raw rings
  uint32_t tmem_base;
  int error;
  int plan[8];               // [0] cache length, [1] first static tile, [2] tiles this CTA streamed, [6] reduction epoch
  int tile_id[16];           // ring: tile streamed as this CTA's i-th (index i & 15), -1 = end of stream
  int page_id[16];           // paged cache: the physical page of that tile
  int stop[4];               // (two used; four keep the 16-byte alignment of what follows) per softmax group: leave the tile loop (end of stream or a wait that ran out)
  int row_lo[NQ], row_hi[NQ];
  float colmax[2][4][NQ];    // per tile parity, per softmax warp
  alignas(16) float bcast[4][2][NQ];     // per softmax warp: minus the reference (0 if -inf), correction factor
  float lsum[4][NQ];
  float mfinal[NQ];
};

static_assert(sizeof(TcCtrl<32>) <= TcCfg<32, 3, 3>::kCtrlBytes && sizeof(TcCtrl<64>) <= TcCfg<64, 2, 3>::kCtrlBytes,
              "control block must fit its shared-memory share");
static_assert(offsetof(TcCtrl<32>, bcast) % 16 == 0 && offsetof(TcCtrl<64>, bcast) % 16 == 0, "bcast is read as float4");

template <int NQ, int NK, int NV, bool FP8 = false>
__global__ void __launch_bounds__(TcCfg<NQ, NK, NV, FP8>::kThreads, 1)
attend_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmKn, const __grid_constant__ CUtensorMap tmVn, const AttendParams p) {
  using C = TcCfg<NQ, NK, NV, FP8>;
  constexpr int D = 128;
  constexpr int kDeq = C::kDeqWarps;   // FP8: converting warps; an operand tile is complete when all have arrived
  constexpr float kNegInf = -INFINITY;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* pipe = smem;                       // K ring, then V ring
  uint8_t* k_ring = smem;
  uint8_t* v_ring = smem + C::kKRingBytes;
  uint8_t* k8_ring = smem + C::kKRingBytes + C::kVRingBytes;        // FP8 only
  uint8_t* v8_ring = k8_ring + C::kRaw * C::kRawTileBytes;
  uint8_t* q_smem = smem + C::kPipeBytes;
  uint8_t* p_smem = q_smem + C::kQBytes;
  TcCtrl<NQ>* ctl = reinterpret_cast<TcCtrl<NQ>*>(p_smem + 2 * C::kQBytes);

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int n_rows = p.n_q * p.G;

#ifdef MASW_TRACE
  long long* tr = p.trace ? p.trace + (static_cast<size_t>((blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x)) * kTraceWords : nullptr;
#endif
  MASW_STAMP(tr, 0);
  // producer state (thread 0 only): the schedule and the pool claim in flight
  constexpr int kStaticNum = 1, kStaticDen = 4;   // share of the tiles that is assigned statically
  constexpr int kHintStatic = 1;                  // statically assigned tiles per CTA named in the next call's L2 hint
  int n_static = 0, static_first = 0, n_pool = 0, n_early = 0, pending = 0x7fffffff;
  int* pool_ctr = nullptr;
  // ---- prologue
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&ctl->tmem_base)),
                 "r"(C::kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (tid == 0) {
    prefetch_tensormap(&tmK);   // the descriptor fetches overlap the barrier setup and the counter loads
    prefetch_tensormap(&tmV);
    // thread 0 is the TMA producer: it initialises the barriers, plans this CTA's tile range and puts
    // the first ring of tiles in flight before the CTA-wide barrier, so that the first HBM round trip
    // overlaps the rest of the prologue (Q tile, TMEM allocation)
    // an operand tile is complete when TMA has delivered it, or (FP8) when both converting warps have written their half
    for (int s = 0; s < NK; ++s) { mbar_init(&ctl->k_full[s], FP8 ? kDeq : 1); mbar_init(&ctl->k_empty[s], 1); }
    for (int s = 0; s < NV; ++s) { mbar_init(&ctl->v_full[s], FP8 ? kDeq : 1); mbar_init(&ctl->v_empty[s], 1); }
    if (FP8) {
      for (int s = 0; s < C::kRaw; ++s) {
        mbar_init(&ctl->k8_full[s], 1); mbar_init(&ctl->k8_empty[s], kDeq);
        mbar_init(&ctl->v8_full[s], 1); mbar_init(&ctl->v8_empty[s], kDeq);
      }
    }
    for (int s = 0; s < 2; ++s) { mbar_init(&ctl->s_full[s], 1); mbar_init(&ctl->s_empty[s], 128 * C::kSoftGroups); }
    for (int s = 0; s < 2; ++s) { mbar_init(&ctl->p_full[s], 128 * C::kSoftGroups); mbar_init(&ctl->p_empty[s], 1); }
    mbar_init(&ctl->o_ready, 1);
    fence_mbar_init();
  }
  // The CTA's first tile is tile number `split`, whatever the cache length turns out to be: it is requested
  // before the length and the epoch have been loaded, which takes their round trip off the path to the first
  // scores.  Should the cache be shorter than that, the tile is streamed all the same and fully masked.
  // When the caller vouches that the kernel in front of this launch writes nothing of K and V (p.early), the
  // request goes out before the wait: a CTA that starts while the predecessor's last CTAs are still draining
  // then has its first tile on the way when the wait ends.
  bool first_requested = false;
  auto request_first_tile = [&](bool with_v = true) {
    const uint64_t policy = l2_policy_evict_first();
    // contiguous cache: tile t of sequence b starts at entry 128 t; paged cache: it is page page_table[b][t]
    // of the pool (the map's outermost coordinate), entries 0..127 of that page
    int row0 = split * C::kTile, outer = b;
    if (p.page_table != nullptr) {
      outer = __ldg(p.page_table + static_cast<size_t>(b) * p.max_pages + split);
      row0 = 0;
      ctl->page_id[0] = outer;
    }
    if (FP8) {
      mbar_arrive_expect_tx(&ctl->k8_full[0], C::kRawTileBytes);
      tma_load_4d(k8_ring, &tmK, &ctl->k8_full[0], 0, row0, kvh, outer, policy);
      mbar_arrive_expect_tx(&ctl->v8_full[0], C::kRawTileBytes);
      tma_load_4d(v8_ring, &tmV, &ctl->v8_full[0], 0, row0, kvh, outer, policy);
    } else {
      mbar_arrive_expect_tx(&ctl->k_full[0], C::kTileBytes);
      tma_load_4d(k_ring, &tmK, &ctl->k_full[0], 0, row0, kvh, outer, policy);
      tma_load_4d(k_ring + C::kSubBytes, &tmK, &ctl->k_full[0], 64, row0, kvh, outer, policy);
      if (with_v) {
        mbar_arrive_expect_tx(&ctl->v_full[0], C::kTileBytes);
        tma_load_4d(v_ring, &tmV, &ctl->v_full[0], 0, row0, kvh, outer, policy);
        tma_load_4d(v_ring + C::kSubBytes, &tmV, &ctl->v_full[0], 64, row0, kvh, outer, policy);
      }
    }
    ctl->tile_id[0] = split;
    n_early = 1;
    first_requested = true;
  };
  // The tile schedule behind the first tile depends on the cache length alone (see the plan below).
  auto plan_schedule = [&](int len) {
    const int nt = (len + C::kTile - 1) / C::kTile;
    const int rest = max(0, nt - p.splits);
    if (p.deterministic) {
      const int base = rest / p.splits, rem = rest % p.splits;
      n_static = base + (split < rem ? 1 : 0);
      n_pool = 0;
      static_first = p.splits + split * base + min(split, rem);
    } else {
      n_static = (rest * kStaticNum / kStaticDen) / p.splits;
      n_pool = rest - n_static * p.splits;
      static_first = p.splits + n_pool + split * n_static;
    }
  };
  int len_early = -1;   // a stable cache includes its length: read ahead of the wait
  if (tid == 0 && p.early && p.page_table == nullptr) {
    constexpr bool kRingEarly = !FP8 && NQ == 32;   // (the 64-row instance is bound by its softmax loop: there the early requests gained nothing)
    request_first_tile(!kRingEarly);   // ring early: only K goes out here, the first V tile follows the Q loads (it is needed a tile later)
    if (kRingEarly) len_early = min(max(__ldg(p.kv_len + b), 0), p.capacity);
  }
  // nothing else above touched global memory: a launch that was allowed to start early waits here for its
  // predecessor, and lets its own successor be set up
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  MASW_STAMP(tr, 10);
  if (tid == 0 && !first_requested) request_first_tile();
  // Everything this thread reads from global memory in the prologue is requested here, back to back, before any
  // of it is used: the cache length, the reduction epoch and the thread's chunks of the Q tile then cost one
  // round trip together instead of one each (thread 0 used to walk three dependent round trips).
  constexpr int kChunksPerRow = D / 8;
  constexpr int kQPerThread = (NQ * kChunksPerRow + C::kThreads - 1) / C::kThreads;
  uint4 qv[kQPerThread];
#pragma unroll
  for (int k = 0; k < kQPerThread; ++k) {
    const int idx = tid + k * C::kThreads;
    const int r = idx / kChunksPerRow, cg = idx % kChunksPerRow;
    qv[k] = make_uint4(0, 0, 0, 0);
    if (idx < NQ * kChunksPerRow && r < n_rows) {
      const int j = r / p.G, g = r % p.G;
      qv[k] = __ldg(reinterpret_cast<const uint4*>(p.q + ((static_cast<size_t>(b) * p.n_q + j) * p.Hq + kvh * p.G + g) * D + cg * 8));
    }
  }
  const int len_raw = (tid < NQ) ? __ldg(p.kv_len + b) : 0;
  const int epoch_raw = (tid == 0) ? __ldcg(p.tickets + (b * p.Hkv + kvh) * (kMaxSplitsDev + 1)) : 0;
  if (tid == 0 && len_early >= 0) {
    // The rest of the K and V rings (this CTA's first static tiles) is requested now, behind the Q loads in the
    // queues but without waiting for them: the prologue's own loads take about 2 us behind the launch's burst of
    // first tiles, and HBM has little else to do meanwhile.
    plan_schedule(len_early);
    const uint64_t policy = l2_policy_evict_first();
    mbar_arrive_expect_tx(&ctl->v_full[0], C::kTileBytes);
    tma_load_4d(v_ring, &tmV, &ctl->v_full[0], 0, split * C::kTile, kvh, b, policy);
    tma_load_4d(v_ring + C::kSubBytes, &tmV, &ctl->v_full[0], 64, split * C::kTile, kvh, b, policy);
    const int n_pre = min((NK < NV ? NK : NV) - 1, n_static);
    for (int i = 1; i <= n_pre; ++i) {
      const int row0 = (static_first + i - 1) * C::kTile;
      uint8_t* kdst = k_ring + i * C::kTileBytes;
      uint8_t* vdst = v_ring + i * C::kTileBytes;
      mbar_arrive_expect_tx(&ctl->k_full[i], C::kTileBytes);
      tma_load_4d(kdst, &tmK, &ctl->k_full[i], 0, row0, kvh, b, policy);
      tma_load_4d(kdst + C::kSubBytes, &tmK, &ctl->k_full[i], 64, row0, kvh, b, policy);
      mbar_arrive_expect_tx(&ctl->v_full[i], C::kTileBytes);
      tma_load_4d(vdst, &tmV, &ctl->v_full[i], 0, row0, kvh, b, policy);
      tma_load_4d(vdst + C::kSubBytes, &tmV, &ctl->v_full[i], 64, row0, kvh, b, policy);
      ctl->tile_id[i] = static_first + i - 1;
    }
    n_early = 1 + n_pre;
  }
  if (tid == 0) {
    const int len = min(max(len_raw, 0), p.capacity);
    // Tile schedule of the tiles behind the first `splits` ones.  A quarter of them is assigned statically
    // (n_static consecutive tiles per split, at the end of the cache, so that the ragged and masked last tile
    // is never the last one a CTA meets); the others form a pool from which the splits of this (sequence,
    // KV head) claim one tile at a time (an atomic counter), so an SM that streams more slowly simply ends up
    // with fewer tiles.  The two counter words alternate with the epoch's parity: this launch uses one, and
    // split 0 clears the other for the next launch, which nobody is using then.
    // In the deterministic mode there is no pool: every tile is assigned statically (the remainder goes to the
    // first splits), so each split meets the same tiles in the same order in every launch and the result
    // repeats bit for bit, at the price of waiting for the slowest SM.
    plan_schedule(len);
    const int epoch = epoch_raw;
    pool_ctr = p.tickets + (b * p.Hkv + kvh) * (kMaxSplitsDev + 1) + 1 + (epoch & 1);
    pending = (n_pool > 0) ? atomicAdd(pool_ctr, 1) : 0x7fffffff;   // used only after the static tiles
    ctl->plan[0] = len;
    ctl->plan[1] = static_first;
    ctl->plan[2] = 0;
    ctl->plan[6] = epoch;
    ctl->error = 0;
    ctl->stop[0] = 0;
    ctl->stop[1] = 0;
  }
  if (tid < NQ) {
    // row j of the T new tokens sees cache entries [0, len - T + j]; padding rows copy the last real row
    const int len = min(max(len_raw, 0), p.capacity);
    const int r = min(tid, n_rows - 1);
    ctl->row_lo[tid] = 0;
    ctl->row_hi[tid] = min(len - p.n_q + r / p.G, len - 1);
  }
#pragma unroll
  for (int k = 0; k < kQPerThread; ++k) {
    const int idx = tid + k * C::kThreads;
    if (idx < NQ * kChunksPerRow) {
      const int r = idx / kChunksPerRow, cg = idx % kChunksPerRow;
      if (FP8) {   // the MMAs run on fp16 operands: q is rounded from bf16 to fp16 (exact but for values below 2^-14)
        uint32_t* w = reinterpret_cast<uint32_t*>(&qv[k]);
#pragma unroll
        for (int e = 0; e < 4; ++e) w[e] = pack_f16x2(__uint_as_float(w[e] << 16), __uint_as_float(w[e] & 0xffff0000u));
      }
      *reinterpret_cast<uint4*>(q_smem + (cg >> 3) * C::kQSubBytes + r * 128 + (((cg & 7) ^ (r & 7)) << 4)) = qv[k];
    }
  }
  fence_proxy_async();   // the Q tile was written with ordinary stores and is read by the tensor core
  tc_fence_before();
  __syncthreads();
  tc_fence_after();

  MASW_STAMP(tr, 1);
  const uint32_t tmem_base = ctl->tmem_base;
  const int kv_total = ctl->plan[0];
  int n_tiles = 0;   // tiles this CTA streamed; each role learns it when it meets the end of the stream
  const uint32_t tmem_o = tmem_base + 2 * NQ;          // columns [2 NQ, 3 NQ): O^T

  if (warp == 0) {
    // ================= TMA producer =================
    if (lane == 0) {
      // Two rings with their own progress: whichever has a free slot gets its next tile (a K slot frees
      // when S^T of its tile is computed, a V slot only when P.V has consumed it).  The polling is bounded.
      // The tile streamed as this CTA's i-th is resolved when the first of the two rings reaches index i
      // (static range first, then pool claims) and recorded in ctl->tile_id for the other warps.  The
      // end of the stream travels through the K ring as an empty "tile" (-1) whose barrier the producer
      // completes itself.
      const uint64_t policy = l2_policy_evict_first();
      int n_res = n_early;   // indices resolved so far (the prologue recorded these)
      auto resolve = [&](int i) -> int {
        if (i < n_res) return ctl->tile_id[i & 15];
        int id = -1;
        if (i - 1 < n_static) {               // index 0 was the first tile, requested in the prologue
          id = static_first + (i - 1);
        } else if (pending < n_pool) {
          id = p.splits + pending;
          pending = atomicAdd(pool_ctr, 1);   // the next claim is in flight while this tile streams
        }
        ctl->tile_id[i & 15] = id;
        if (p.page_table != nullptr && id >= 0)
          ctl->page_id[i & 15] = __ldg(p.page_table + static_cast<size_t>(b) * p.max_pages + id);
        n_res = i + 1;
        return id;
      };
      int ik = n_early, iv = n_early;   // the first tiles were issued in the prologue
      bool k_done = false, v_done = false;
      int idle = 0;
      while ((!k_done || !v_done) && idle < MASW_WAIT_LIMIT(p)) {
        bool progressed = false;
        // (FP8: the producer fills the raw rings; the converting warps fill the operand buffers from them)
        constexpr int RK = FP8 ? C::kRaw : NK, RV = FP8 ? C::kRaw : NV;
        uint64_t* const kf = FP8 ? ctl->k8_full : ctl->k_full;
        uint64_t* const ke = FP8 ? ctl->k8_empty : ctl->k_empty;
        uint64_t* const vf = FP8 ? ctl->v8_full : ctl->v_full;
        uint64_t* const ve = FP8 ? ctl->v8_empty : ctl->v_empty;
        if (!k_done && (ik < RK || mbar_try_wait(&ke[ik % RK], (ik / RK - 1) & 1))) {
          const int id = resolve(ik);
          if (id < 0) {
            mbar_arrive(&kf[ik % RK]);
            k_done = true;
          } else {
            const bool paged = p.page_table != nullptr;
            const int row0 = paged ? 0 : id * C::kTile, outer = paged ? ctl->page_id[ik & 15] : b;
            mbar_arrive_expect_tx(&kf[ik % RK], FP8 ? C::kRawTileBytes : C::kTileBytes);
#ifdef MASW_TRACE
            if (ik != p.drop_tile)
#endif
            {
              if (FP8) {
                tma_load_4d(k8_ring + (ik % RK) * C::kRawTileBytes, &tmK, &kf[ik % RK], 0, row0, kvh, outer, policy);
              } else {
                uint8_t* kdst = k_ring + (ik % NK) * C::kTileBytes;
                tma_load_4d(kdst, &tmK, &kf[ik % RK], 0, row0, kvh, outer, policy);
                tma_load_4d(kdst + C::kSubBytes, &tmK, &kf[ik % RK], 64, row0, kvh, outer, policy);
              }
            }
            ++ik;
          }
          progressed = true;
        }
        if (!v_done && (iv < RV || mbar_try_wait(&ve[iv % RV], (iv / RV - 1) & 1))) {
          const int id = resolve(iv);
          if (id < 0) {
            v_done = true;
          } else {
            const bool paged = p.page_table != nullptr;
            const int row0 = paged ? 0 : id * C::kTile, outer = paged ? ctl->page_id[iv & 15] : b;
            mbar_arrive_expect_tx(&vf[iv % RV], FP8 ? C::kRawTileBytes : C::kTileBytes);
            if (FP8) {
              tma_load_4d(v8_ring + (iv % RV) * C::kRawTileBytes, &tmV, &vf[iv % RV], 0, row0, kvh, outer, policy);
            } else {
              uint8_t* vdst = v_ring + (iv % NV) * C::kTileBytes;
              tma_load_4d(vdst, &tmV, &vf[iv % RV], 0, row0, kvh, outer, policy);
              tma_load_4d(vdst + C::kSubBytes, &tmV, &vf[iv % RV], 64, row0, kvh, outer, policy);
            }
            ++iv;
          }
          progressed = true;
        }
        idle = progressed ? 0 : idle + 1;
        if (!progressed) __nanosleep(64);   // leave the issue slots of this scheduler to the softmax warps
      }
      if (!k_done || !v_done) ctl->error = 1;
      ctl->plan[2] = iv;
      // Every tile of this launch is requested: ask for the tile this CTA will stream first in the NEXT call (the
      // next layer's cache, same geometry) to be brought into L2.  The requests queue behind this CTA's own last
      // tiles and land while the launch is in its reduction, so the next launch's first tile is an L2 hit.
      if (p.next_hint) {
        tma_prefetch_4d(&tmKn, 0, split * C::kTile, kvh, b);
        tma_prefetch_4d(&tmKn, 64, split * C::kTile, kvh, b);
        tma_prefetch_4d(&tmVn, 0, split * C::kTile, kvh, b);
        tma_prefetch_4d(&tmVn, 64, split * C::kTile, kvh, b);
        // ... and its statically assigned tiles, which it streams next (the same numbers when the next cache is as
        // long): HBM is idle while this launch publishes and reduces, and these bytes then need not cross it again
        for (int i = 0; i < min(n_static, kHintStatic); ++i) {
          const int row0 = (static_first + i) * C::kTile;
          tma_prefetch_4d(&tmKn, 0, row0, kvh, b);
          tma_prefetch_4d(&tmKn, 64, row0, kvh, b);
          tma_prefetch_4d(&tmVn, 0, row0, kvh, b);
          tma_prefetch_4d(&tmVn, 64, row0, kvh, b);
        }
      }
    }
  } else if (warp == 1) {
    // ================= MMA issuer =================
    if (lane == 0) {
      constexpr uint32_t idesc1 = tc_idesc(128, NQ, 0, 0, FP8);   // K (K-major) x Q (K-major)
      // V^T (MN-major) x P (MN-major too: [entry][row], one line of NQ rows per entry, 128 bytes with the 128B
      // swizzle or 64 bytes with the 64B swizzle, so that a softmax thread, which owns an entry, writes its
      // probabilities as 16-byte chunks of its own line)
      constexpr uint32_t idesc2 = tc_idesc(128, NQ, 1, 1, FP8);
      const uint32_t q_base = smem_u32(q_smem), p_base = smem_u32(p_smem);
      bool ok = true;
      int n_end = 0x7fffffff;   // index of the end-of-stream marker, once met
      for (int i = 0; ok; ++i) {
        {
          const int sb = i & 1;
          ok = mbar_wait_bounded(&ctl->k_full[i % NK], (i / NK) & 1, MASW_WAIT_LIMIT(p));
          if (ok && i >= 2) ok = mbar_wait_bounded(&ctl->s_empty[sb], ((i >> 1) - 1) & 1, MASW_WAIT_LIMIT(p));
          if (!ok) break;
          if (ctl->tile_id[i & 15] < 0) {
            n_end = i;
            mbar_arrive(&ctl->s_full[sb]);   // hands the end of the stream on to the softmax warps
          } else {
            tc_fence_after();
            const uint32_t k_base = smem_u32(k_ring + (i % NK) * C::kTileBytes);
#pragma unroll
            for (int ks = 0; ks < D / 16; ++ks) {
              const uint32_t off = (ks >> 2) * C::kSubBytes + (ks & 3) * 32;
              const uint32_t qoff = (ks >> 2) * C::kQSubBytes + (ks & 3) * 32;
              tc_mma_bf16(tmem_base + sb * NQ, tc_desc_kmajor(k_base + off), tc_desc_kmajor(q_base + qoff), idesc1, ks > 0);
            }
            tc_commit(&ctl->s_full[sb]);
            tc_commit(&ctl->k_empty[i % NK]);   // the K tile is no longer needed once S^T is computed
          }
        }
        if (i >= 1) {
          const int j = i - 1;
          ok = mbar_wait_bounded(&ctl->p_full[j & 1], (j >> 1) & 1, MASW_WAIT_LIMIT(p));
          if (ok) ok = mbar_wait_bounded(&ctl->v_full[j % NV], (j / NV) & 1, MASW_WAIT_LIMIT(p));
          if (!ok) break;
          tc_fence_after();
          const uint32_t v_base = smem_u32(v_ring + (j % NV) * C::kTileBytes);
#pragma unroll
          for (int kk = 0; kk < C::kTile / 16; ++kk) {
            const uint32_t poff = (j & 1) * C::kQBytes + kk * 16 * (2 * NQ);   // 16 entries per MMA
            const uint64_t p_desc = NQ == 64 ? tc_desc_mnmajor(p_base + poff, C::kSubBytes) : tc_desc_mnmajor_sw64(p_base + poff);
            tc_mma_bf16(tmem_o, tc_desc_mnmajor(v_base + kk * 2048, C::kSubBytes), p_desc, idesc2,
                        (j > 0 || kk > 0) ? 1u : 0u);
          }
          tc_commit(&ctl->v_empty[j % NV]);   // the V tile of tile j is no longer needed
          tc_commit(&ctl->p_empty[j & 1]);    // this P tile may be overwritten
          tc_commit(&ctl->o_ready);           // O^T includes tile j
        }
        if (i >= n_end) break;
      }
      if (!ok) ctl->error = 1;
    }
  } else if (FP8 && (warp == 2 || warp == 3 || warp >= 12)) {
    // ================= FP8: raw tile -> fp16 operand tile =================
    // Six warps share every K and V tile (groups of four entries, dealt round-robin).  A lane takes one 16-byte chunk
    // (16 e4m3 values of one entry), widens it to fp16 (exact), multiplies by the page's scale in fp16 (one
    // rounding: this product IS the dequantised value the result is defined on) and writes the two 16-byte chunks
    // into the operand tile in the swizzled layout a bf16 tile has.  The end of the stream travels on as it does
    // for the bf16 cache: the producer completes the raw K barrier of an empty "tile", and the warps pass it to
    // the MMA issuer through the operand barrier.
    const int didx = warp < 4 ? warp - 2 : warp - 10;   // 0..5: takes every sixth group of four rows
    const int c = lane & 7;                       // 16-byte chunk of the raw row: dims 16 c .. 16 c + 15
    const int r_in = lane >> 3;                   // row inside a group of four
    bool ok = true;
    auto convert = [&](const uint8_t* raw, uint8_t* dst, uint32_t scale2) {
#ifdef MASW_TRACE
      if (p.debug_flags & 32) return;   // timing experiment: no conversion (results are then meaningless)
#endif
#pragma unroll 3
      for (int it = didx; it < 32; it += kDeq) {
        const int r = it * 4 + r_in;
        const uint4 x = *reinterpret_cast<const uint4*>(raw + r * 128 + ((c ^ (r & 7)) << 4));
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
        uint32_t h[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          h[2 * e] = hmul2_u32(e4m3x2_to_f16x2(w[e] & 0xffffu), scale2);
          h[2 * e + 1] = hmul2_u32(e4m3x2_to_f16x2(w[e] >> 16), scale2);
        }
        uint8_t* row = dst + (c >> 2) * C::kSubBytes + r * 128;
        const int c16 = (c & 3) * 2;
        *reinterpret_cast<uint4*>(row + (((c16) ^ (r & 7)) << 4)) = make_uint4(h[0], h[1], h[2], h[3]);
        *reinterpret_cast<uint4*>(row + (((c16 + 1) ^ (r & 7)) << 4)) = make_uint4(h[4], h[5], h[6], h[7]);
      }
    };
    for (int i = 0; ok; ++i) {
      ok = mbar_wait_bounded(&ctl->k8_full[i % C::kRaw], (i / C::kRaw) & 1, MASW_WAIT_LIMIT(p));
      if (!ok) break;
      const int tile = ctl->tile_id[i & 15];
      if (tile < 0) {   // end of the stream: hand it on to the MMA issuer
        if (i >= NK) ok = mbar_wait_bounded(&ctl->k_empty[i % NK], (i / NK - 1) & 1, MASW_WAIT_LIMIT(p));
        if (lane == 0) mbar_arrive(&ctl->k_full[i % NK]);
        break;
      }
      const int page = ctl->page_id[i & 15];
      const float ks = __ldg(p.k_scale + static_cast<size_t>(page) * p.Hkv + kvh);
      const float vs = __ldg(p.v_scale + static_cast<size_t>(page) * p.Hkv + kvh);
      if (i >= NK) ok = mbar_wait_bounded(&ctl->k_empty[i % NK], (i / NK - 1) & 1, MASW_WAIT_LIMIT(p));
      if (!ok) break;
      convert(k8_ring + (i % C::kRaw) * C::kRawTileBytes, k_ring + (i % NK) * C::kTileBytes, pack_f16x2(ks, ks));
      fence_proxy_async();   // the operand tile was written with ordinary stores and is read by the tensor core
      __syncwarp();
      if (lane == 0) { mbar_arrive(&ctl->k_full[i % NK]); mbar_arrive(&ctl->k8_empty[i % C::kRaw]); }
      ok = mbar_wait_bounded(&ctl->v8_full[i % C::kRaw], (i / C::kRaw) & 1, MASW_WAIT_LIMIT(p));
      if (ok && i >= NV) ok = mbar_wait_bounded(&ctl->v_empty[i % NV], (i / NV - 1) & 1, MASW_WAIT_LIMIT(p));
      if (!ok) break;
      convert(v8_ring + (i % C::kRaw) * C::kRawTileBytes, v_ring + (i % NV) * C::kTileBytes, pack_f16x2(vs, vs));
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) { mbar_arrive(&ctl->v_full[i % NV]); mbar_arrive(&ctl->v8_empty[i % C::kRaw]); }
    }
    if (!ok) ctl->error = 1;
  } else if (warp >= 4 && warp < 12) {
    // ================= softmax warps =================
    // kSoftGroups groups of four warps; group g owns the query rows (TMEM columns) [kCols g, kCols g + kCols), and
    // inside a group thread <-> TMEM lane <-> entry.  Columns are independent, so the groups only share the
    // barriers that hand S^T and P^T over.
    constexpr int kCols = C::kCols;
    const int lc = lane % kCols;                         // the column (of this group) this lane keeps the statistics of
    const int grp = (warp - 4) >> 2;
    const int w = (warp - 4) & 3;
    const int cg = grp * kCols;                          // first column of this group
    const int e = w * 32 + lane;                         // entry inside the tile == TMEM lane
    const uint32_t lane_addr = static_cast<uint32_t>(w * 32) << 16;
    const int bar_id = 1 + grp;
    float m_col = kNegInf;                               // lane c: softmax reference of column cg + c
    float l_part[kCols];
#pragma unroll
    for (int c = 0; c < kCols; ++c) l_part[c] = 0.f;
    // A wait that runs out makes the thread "dead": it stops waiting but keeps walking the loop, so
    // that every thread still meets every named barrier (the results are then meaningless and the
    // status word says so).
    bool ok = true;

    volatile int* stop = &ctl->stop[grp];
    constexpr float kSlack = 8.f;
    bool refs_finite = false;   // every row of the group has a finite reference (identical in the group's threads)
    for (int i = 0;; ++i) {
      const int sb = i & 1;
      bool exceed = false;
      if (ok) ok = mbar_wait_bounded(&ctl->s_full[sb], (i >> 1) & 1, MASW_WAIT_LIMIT(p));
      ok = __all_sync(0xffffffffu, ok);
      const int tile = ctl->tile_id[i & 15];
      // The loop ends for the whole group at the named barrier below: at the end-of-stream marker, or
      // when a wait ran out in any of its warps (the results are then meaningless and the status word
      // says so).  Every thread reaches that barrier in every iteration it starts.
      const bool live = ok && tile >= 0;
      float s[kCols];
      const int x = tile * C::kTile + e;
      const bool tile_masked = ((tile + 1) * C::kTile - 1) > ctl->row_hi[0];   // row 0 has the smallest bound
      if (live) {
        tc_fence_after();
#pragma unroll
        for (int cb = 0; cb < kCols; cb += 16) {
          float v16[16];
          tc_ld16(tmem_base + lane_addr + sb * NQ + cg + cb, v16);
#pragma unroll
          for (int c = 0; c < 16; ++c) s[cb + c] = v16[c];
        }
        tc_wait_ld();
        tc_fence_before();
        mbar_arrive(&ctl->s_empty[sb]);

        // mask: this thread's entry index against each row's visibility bounds (the scores stay unscaled: the
        // positive scale commutes with the maximum and is folded into the exponent's multiply-add)
        if (tile_masked) {
#pragma unroll
          for (int c = 0; c < kCols; ++c) s[c] = (x <= ctl->row_hi[cg + c]) ? s[c] : kNegInf;
        }
        // Does any score of this thread exceed its row's reference by more than the slack?  After the first few
        // tiles the answer is almost always no for all 128 threads of the group, and then the column maxima are
        // not needed at all: the references stay, nothing is rescaled, and the exchange below is skipped.
        if (refs_finite) {
#pragma unroll
          for (int c4 = 0; c4 < kCols; c4 += 4) {
            const float4 mu4 = *reinterpret_cast<const float4*>(&ctl->bcast[w][0][cg + c4]);
            exceed |= fmaf(s[c4], p.scale_log2e, mu4.x) > kSlack || fmaf(s[c4 + 1], p.scale_log2e, mu4.y) > kSlack ||
                      fmaf(s[c4 + 2], p.scale_log2e, mu4.z) > kSlack || fmaf(s[c4 + 3], p.scale_log2e, mu4.w) > kSlack;
          }
        } else {
          exceed = true;   // some row has no finite reference yet
        }
      } else {
        *stop = 1;
      }
      const bool move = named_bar_red_or(bar_id, 128, exceed);
      if (*stop != 0) {
        n_tiles = i;
        break;
      }
      bool any_changed = false;
      if (move) {
      // column maxima over the 128 entries: butterfly inside the warp, then across the group's four warps
      {
        float t[kCols];
#pragma unroll
        for (int c = 0; c < kCols; ++c) t[c] = s[c];
        ctl->colmax[i & 1][w][cg + lc] = warp_transpose_reduce<kCols, true>(t, lane);
      }
      named_bar_sync(bar_id, 128);
      // The reference each column subtracts (m_col) follows the running maximum lazily: it moves only
      // when the new maximum exceeds it by more than kSlack (in log2 units), so probabilities may reach
      // 2^kSlack instead of 1, which bf16 / fp32 hold without loss, and the O^T accumulator in tensor
      // memory has to be rescaled only on those rare moves.  o = O / l is unchanged by the choice.
      bool changed;
      {
        const int c = cg + lc;
        const float mx = fmaxf(fmaxf(ctl->colmax[i & 1][0][c], ctl->colmax[i & 1][1][c]),
                               fmaxf(ctl->colmax[i & 1][2][c], ctl->colmax[i & 1][3][c])) * p.scale_log2e;
        changed = mx > m_col + kSlack;                     // also true for the first finite maximum (-inf + 8)
        const float m_new = changed ? mx : m_col;
        const float mu = (m_new == kNegInf) ? 0.f : m_new;
        ctl->bcast[w][0][c] = -mu;
        ctl->bcast[w][1][c] = changed ? fast_exp2(m_col - mu) : 1.f;
        m_col = m_new;
      }
      any_changed = __any_sync(0xffffffffu, changed);   // identical in the group's four warps
      refs_finite = __all_sync(0xffffffffu, m_col != kNegInf);
      __syncwarp();
      }   // if (move)

      // probabilities (rounded to bf16, the row sums use the rounded values)
      uint32_t pk[kCols / 2];   // packed pairs of consecutive rows
#ifdef MASW_TRACE
      if (p.debug_flags & 64) {   // timing experiment: no exponentials
#pragma unroll
        for (int c = 0; c < kCols / 2; ++c) pk[c] = 0;
      } else
#endif
#pragma unroll
      for (int c4 = 0; c4 < kCols; c4 += 4) {
        const float4 mu4 = *reinterpret_cast<const float4*>(&ctl->bcast[w][0][cg + c4]);
        float4 cr4 = make_float4(1.f, 1.f, 1.f, 1.f);
        if (any_changed) cr4 = *reinterpret_cast<const float4*>(&ctl->bcast[w][1][cg + c4]);
        const float nmu[4] = {mu4.x, mu4.y, mu4.z, mu4.w};   // minus the reference of each row
        const float cr[4] = {cr4.x, cr4.y, cr4.z, cr4.w};
#pragma unroll
        for (int k = 0; k < 4; k += 2) {   // two probabilities per conversion instruction
          const float pv0 = fast_exp2(fmaf(s[c4 + k], p.scale_log2e, nmu[k]));
          const float pv1 = fast_exp2(fmaf(s[c4 + k + 1], p.scale_log2e, nmu[k + 1]));
          const uint32_t pr2 = FP8 ? pack_f16x2(pv0, pv1) : pack_bf16x2(pv0, pv1);
          pk[(c4 + k) >> 1] = pr2;
          l_part[c4 + k] = l_part[c4 + k] * cr[k] + (FP8 ? f16_lo_to_f32(pr2) : __uint_as_float(pr2 << 16));
          l_part[c4 + k + 1] = l_part[c4 + k + 1] * cr[k + 1] + (FP8 ? f16_hi_to_f32(pr2) : __uint_as_float(pr2 & 0xffff0000u));
        }
      }

      // the P tile is double-buffered: tile i - 2's P.V must be complete before its buffer is reused;
      // only a moved maximum has to wait for tile i - 1's P.V, to rescale O^T in tensor memory
      if (i >= 2 && ok) ok = mbar_wait_bounded(&ctl->p_empty[i & 1], ((i >> 1) - 1) & 1, MASW_WAIT_LIMIT(p));
      if (i > 0 && any_changed) {
        if (ok) ok = mbar_wait_bounded(&ctl->o_ready, (i - 1) & 1, MASW_WAIT_LIMIT(p));
        ok = __all_sync(0xffffffffu, ok);   // the tensor-memory accesses below are warp-wide
        tc_fence_after();
        if (ok) {
#pragma unroll
          for (int cb = 0; cb < kCols; cb += 16) {
            float v16[16];
            tc_ld16(tmem_o + lane_addr + cg + cb, v16);
            tc_wait_ld();
#pragma unroll
            for (int c = 0; c < 16; ++c) v16[c] *= ctl->bcast[w][1][cg + cb + c];
            tc_st16(tmem_o + lane_addr + cg + cb, v16);
          }
          tc_wait_st();
        }
      }
      // P -> shared memory as the MN-major B operand [entry e][row]: this thread's rows are consecutive bytes
      // of its entry's line (free of bank conflicts: eight consecutive lines cover all banks under the swizzle)
      {
        uint8_t* pline = p_smem + (i & 1) * C::kQBytes + e * (2 * NQ);
        const int sw = (NQ == 64) ? (e & 7) : ((e >> 1) & 3);   // 128B / 64B swizzle of the 16-byte chunks
#pragma unroll
        for (int q = 0; q < kCols / 8; ++q) {
          const int chunk = (cg >> 3) + q;
          *reinterpret_cast<uint4*>(pline + ((chunk ^ sw) << 4)) = make_uint4(pk[4 * q], pk[4 * q + 1], pk[4 * q + 2], pk[4 * q + 3]);
        }
      }
      // entries beyond the cache length hold foreign bytes: zero their V rows (their probability is 0,
      // but 0 x non-finite would poison the accumulator); the first group does it
      if (grp == 0 && (tile + 1) * C::kTile > kv_total) {   // only the last tile of the cache can have such rows
        if (ok) ok = mbar_wait_bounded(&ctl->v_full[i % NV], (i / NV) & 1, MASW_WAIT_LIMIT(p));   // the tile must have landed before it is patched
        // rows [valid, 128) are one contiguous range in each 64-column half of the tile (the swizzle
        // permutes inside a row group, and whole rows are cleared); consecutive threads clear
        // consecutive 16-byte chunks, which is free of bank conflicts
        const int valid = max(0, kv_total - tile * C::kTile);   // a first tile beyond the cache has no valid row
        uint8_t* vt = v_ring + (i % NV) * C::kTileBytes;
        for (int idx = valid * 8 + e; idx < C::kTile * 8; idx += 128) {
          *reinterpret_cast<uint4*>(vt + idx * 16) = make_uint4(0, 0, 0, 0);
          *reinterpret_cast<uint4*>(vt + C::kSubBytes + idx * 16) = make_uint4(0, 0, 0, 0);
        }
      }
      fence_proxy_async();
      tc_fence_before();
      mbar_arrive(&ctl->p_full[i & 1]);
    }
    if (!ok) ctl->error = 1;
    MASW_STAMP_BY(tr, 128, 8);

    // ---- epilogue of the softmax warps: this split's partial (o unnormalised, m, l) -> global scratch
    const int bh = b * p.Hkv + kvh;
    unsigned long long* po = p.part_o + (static_cast<size_t>(bh) * p.splits + split) * NQ * D;
    unsigned long long* pml = p.part_ml + (static_cast<size_t>(bh) * p.splits + split) * NQ * 2;
    const int tag = ctl->plan[6] + 1;   // this launch's epoch tag
    bool have_o = ok && n_tiles > 0;
    if (have_o) {
      have_o = mbar_wait_bounded(&ctl->o_ready, (n_tiles - 1) & 1, MASW_WAIT_LIMIT(p));
      tc_fence_after();
    }
    have_o = __all_sync(0xffffffffu, have_o);
    {
      float t[kCols];
#pragma unroll
      for (int c = 0; c < kCols; ++c) t[c] = l_part[c];
      ctl->lsum[w][cg + lc] = warp_transpose_reduce<kCols, false>(t, lane);
      if (w == 0) ctl->mfinal[cg + lc] = m_col;
    }
#pragma unroll
    for (int cb = 0; cb < kCols; cb += 16) {
      float v16[16];
      if (have_o) {
        tc_ld16(tmem_o + lane_addr + cg + cb, v16);
        tc_wait_ld();
      } else {
#pragma unroll
        for (int c = 0; c < 16; ++c) v16[c] = 0.f;
      }
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        if (cg + cb + c < n_rows) rec_store1(po + (cg + cb + c) * D + e, v16[c], tag);   // thread e holds dimension e of every row
      }
    }
    named_bar_sync(bar_id, 128);
    if (e < kCols && cg + e < n_rows) {
      const int r = cg + e;
      rec_store2(pml + r * 2, ctl->mfinal[r], ctl->lsum[0][r] + ctl->lsum[1][r] + ctl->lsum[2][r] + ctl->lsum[3][r], tag);
    }
    tc_fence_before();
    MASW_STAMP_BY(tr, 128, 9);
  }

  __syncthreads();
  MASW_STAMP(tr, 2);
#ifdef MASW_TRACE
  if (tr && tid == 0) { tr[6] = ctl->plan[2]; unsigned sm; asm("mov.u32 %0, %%smid;" : "=r"(sm)); tr[7] = sm; }
#endif
  if (ctl->error != 0) {
    if (tid == 0 && p.status) atomicOr(p.status, MASW_STATUS_WAIT_TIMEOUT);
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::kTmemCols) : "memory");
  }
  MASW_STAMP(tr, 3);
  // six thread groups per item with three splits' records in flight each: 18 splits in one round trip, and few
  // enough registers that nothing spills
  // (the 64-row instance has up to 114 items per CTA: three groups x six records take them in one batch, and its
  // 168-register cap has room for the eighteen records in flight)
  constexpr int kRG = FP8 ? 8 : (NQ == 64 ? 3 : 6), kRF = (!FP8 && NQ == 64) ? 6 : 3;
  static_assert(C::kThreads % kRG == 0, "the fetch groups must divide the thread count");
  split_reduce_and_store<D, NQ, C::kThreads, kRG, kRF>(p, b, kvh, split, n_rows, ctl->plan[6], reinterpret_cast<float*>(pipe), tid);
  // the pool counter of the next launch (the other parity) is idle now: clear it
  if (split == 0 && tid == 0) p.tickets[(b * p.Hkv + kvh) * (kMaxSplitsDev + 1) + 1 + ((ctl->plan[6] + 1) & 1)] = 0;
  MASW_STAMP(tr, 4);
}

}  // namespace masw
