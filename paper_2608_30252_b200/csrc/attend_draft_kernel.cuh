// Draft decode attention for up to eight query rows per KV head (one or two tokens x a group of <= 8 heads):
// the launch that a draft step repeats once per layer, where latency, not bandwidth, is what a batch-1 decode
// pays for.  Same split-K skeleton and the same cross-split reduction as attend_kernel, with three changes:
//
//  * Footprint.  113 KB of shared memory (seven 16 KB stages) and <= 128 registers x 256 threads, so that two
//    CTAs fit on an SM: with programmatic dependent launch the CTAs of layer l + 1 become resident while layer
//    l's are still in their reduction.
//  * Order.  What does not depend on the predecessor runs ABOVE griddepcontrol.wait when the host says so
//    (AttendParams::early): the counters, the plan and the bulk copies of this layer's K/V tiles, which the
//    predecessor (another layer's launch) does not write.  Below the wait only q, the pending raw K/V rows and
//    the reduction epoch are read; by then the tiles are already in shared memory.
//  * Orientation.  The tensor-core M dimension is given to the ENTRIES and the (padded) eight query rows are
//    N: S^T[16 entries x 8 rows] = K . Q^T and O^T[16 dims x 8 rows] += V^T . P^T with mma.sync.m16n8k16, half
//    the instructions of the rows-on-M form, and no query tile in shared memory: the Q^T fragments are loaded
//    from global memory straight into registers.  P^T reaches its operand layout with movmatrix; it is carried
//    as hi + lo bf16 terms, which removes the bf16 rounding of the probabilities from the result.
//
// All eight warps consume: warp w owns tiles w, w + 8, ...  There is no producer warp: thread 0 requests the first
// seven tiles, and the warp that has consumed tile i requests tile i + 7 into the stage it just freed.  A stage
// is therefore met by different warps in different rounds: before it tests a barrier phase a warp checks
// that the stage has been re-armed for its tile (a word per stage in shared memory), which keeps the parity
// test from aliasing with an older phase.
#pragma once

#include "attend_kernel.cuh"

namespace masw {

template <int D>
struct DraftCfg {
  static constexpr int kWarps = 8;                          // all of them consume
  static constexpr int kThreads = kWarps * 32;
  static constexpr int kRows = 8;                           // query rows (padded)
  static constexpr int TE = (D == 64) ? 64 : 32;            // entries per tile
  static constexpr int kSub = D / 64;                       // 128-byte column groups
  static constexpr int kSubBytes = TE * 128;                // one [TE x 64] bf16 box
  static constexpr int kTileBytes = kSub * kSubBytes;       // K or V tile: 8 KB
  static constexpr int kStageBytes = 2 * kTileBytes;        // 16 KB
  static constexpr int kStages = 7;
  static constexpr int kPipeBytes = kStages * kStageBytes;  // 112 KB
  static constexpr int kCtrlBytes = 1024;
  static constexpr int kSmemBytes = kPipeBytes + kCtrlBytes;   // 113 KB: two CTAs (and their 1 KB reserves) fill an SM's 228 KB
  static constexpr int kMergeStride = D + 8;                // floats per partial row in shared memory
  // scratch that reuses the stages once every tile is consumed
  static constexpr int kMergeOff = 0;                                        // [kWarps][kRows][kMergeStride] + [kWarps][kRows][2]
  static constexpr int kMergeBytes = kWarps * kRows * (kMergeStride + 2) * 4;
  static constexpr int kProjHsOff = 40 * 1024;                               // slot projection: hidden-state slice (<= 16 KB)
  static constexpr int kProjRedOff = 56 * 1024;                              // [row lanes][2 D] partial sums (<= 18 KB)
  static constexpr int kRopeOff = 80 * 1024;                                 // [D/2][2] doubles
  static constexpr int kReduceOff = 84 * 1024;                               // scratch of split_reduce_and_store
  static_assert(D == 64 || D == 128, "head_dim");
  static_assert(kMergeBytes <= kProjHsOff, "merge scratch overlaps the projection staging");
  static_assert(kReduceOff + kThreads * 24 + 8 * D + 64 <= kPipeBytes, "reduction scratch must fit in the stages");
  static_assert(kSmemBytes <= 113 * 1024, "two CTAs per SM");
};

struct DraftCtrl {
  uint64_t full_bar[8];
  int plan[48];        // [0] nseg, [1] tile_begin, [2] tile_end, [3] error flag, [6] reduction epoch, [7] committed tokens t,
                       // [8 + 4 s ..] phys, len, xbase, kind of segment s, [32 + s] first tile of segment s (s = 0..nseg)
  int row_lo[kMaxSeg * 8], row_hi[kMaxSeg * 8];
  int armed[8];        // per stage: 1 + the CTA-local index of the tile the stage was last armed (and requested) for
};
static_assert(sizeof(DraftCtrl) <= 1024, "control block");

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

__device__ __forceinline__ int ld_acquire_shared(const int* p) {
  int v;
  asm volatile("ld.acquire.cta.shared.b32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
  return v;
}
__device__ __forceinline__ void st_release_shared(int* p, int v) {
  asm volatile("st.release.cta.shared.b32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}

template <int D>
__global__ void __launch_bounds__(DraftCfg<D>::kThreads, 2)
attend_draft_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const AttendParams p) {
  using C = DraftCfg<D>;
  constexpr int TE = C::TE;
  constexpr int NW = C::kWarps;
  constexpr int NS = C::kStages;
  constexpr float kNegInf = -INFINITY;

  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* pipe = smem_raw;   // the dynamic shared memory of a kernel without static shared memory starts 1 KB aligned
  DraftCtrl* ctl = reinterpret_cast<DraftCtrl*>(smem_raw + C::kPipeBytes);
  int* plan = ctl->plan;

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int n_rows = p.n_q * p.G;   // real query rows of this KV head (<= 8)
  const bool is_producer = (tid == 0);   // requests the first ring of tiles

#ifdef MASW_TRACE
  long long* tr = p.trace ? p.trace + (static_cast<size_t>((blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x)) * kTraceWords : nullptr;
#endif
  MASW_STAMP(tr, 0);

  if (is_producer) {
    prefetch_tensormap(&tmK);
    prefetch_tensormap(&tmV);
    for (int s = 0; s < NS; ++s) mbar_init(&ctl->full_bar[s], 1);
    fence_mbar_init();
  }

  // ---- plan (segments, this CTA's tile range, per-row visibility bounds) and the first ring of copies.
  // It reads only the counters and requests only this layer's K/V: with p.early it runs before the wait.
  auto plan_and_issue = [&]() {
    Segment seg[kMaxSeg];
    int t_b, m_b;
    const int nseg = build_segments(p, b, seg, t_b, m_b);
    if (tid == 0) {
      int acc = 0;
      for (int s = 0; s < nseg; ++s) {
        plan[8 + 4 * s + 0] = seg[s].phys;
        plan[8 + 4 * s + 1] = seg[s].len;
        plan[8 + 4 * s + 2] = seg[s].xbase;
        plan[8 + 4 * s + 3] = seg[s].kind;
        plan[32 + s] = acc;
        acc += (seg[s].len + TE - 1) / TE;
      }
      plan[32 + nseg] = acc;
      plan[0] = nseg;
      plan[1] = static_cast<int>((static_cast<long long>(acc) * split) / p.splits);
      plan[2] = static_cast<int>((static_cast<long long>(acc) * (split + 1)) / p.splits);
      plan[3] = 0;
      plan[7] = t_b;
    }
    if (is_producer) {
      int first[kMaxSeg + 1];
      int acc = 0;
      for (int s = 0; s < nseg; ++s) { first[s] = acc; acc += (seg[s].len + TE - 1) / TE; }
      first[nseg] = acc;
      const int tb = static_cast<int>((static_cast<long long>(acc) * split) / p.splits);
      const int te = static_cast<int>((static_cast<long long>(acc) * (split + 1)) / p.splits);
      const uint64_t policy = l2_policy_evict_first();
      const int n0 = min(te - tb, NS);
      int sg = 0;
      for (int i = 0; i < n0; ++i) {
        const int it = tb + i;
        while (sg + 1 < nseg && it >= first[sg + 1]) ++sg;
        const int row0 = seg[sg].phys + (it - first[sg]) * TE;
        uint8_t* kdst = pipe + i * C::kStageBytes;
        uint8_t* vdst = kdst + C::kTileBytes;
        mbar_arrive_expect_tx(&ctl->full_bar[i], C::kStageBytes);
#ifdef MASW_TRACE
        if (i == p.drop_tile) continue;
#endif
#pragma unroll
        for (int sub = 0; sub < C::kSub; ++sub)
          tma_load_4d(kdst + sub * C::kSubBytes, &tmK, &ctl->full_bar[i], sub * 64, row0, kvh, b, policy);
#pragma unroll
        for (int sub = 0; sub < C::kSub; ++sub)
          tma_load_4d(vdst + sub * C::kSubBytes, &tmV, &ctl->full_bar[i], sub * 64, row0, kvh, b, policy);
      }
      for (int s = 0; s < NS; ++s) ctl->armed[s] = (s < n0) ? s + 1 : 0;
    }
    if (tid < C::kRows) {
      const int r = min(tid, n_rows - 1);
      const int j = r / p.G;
      const int n_raw = p.n_q - p.last_row_is_slot;
      const bool is_slot = p.last_row_is_slot && (j == p.n_q - 1);
      const int last = t_b + (is_slot ? n_raw - 1 : j);
      const int lo_raw = max(p.S, last + 1 - p.W);
      const int hi_raw = last;
      const int hi_slot = m_b - 1 + ((is_slot && p.h_g == nullptr) ? 1 : 0);
      for (int s = 0; s < kMaxSeg; ++s) {
        int lo = 1, hi = 0;
        if (s < nseg) {
          const int x_first = seg[s].xbase, x_last = seg[s].xbase + seg[s].len - 1;
          if (seg[s].kind == 0) { lo = 0; hi = hi_raw; }
          else if (seg[s].kind == 1) { lo = 0; hi = hi_slot; }
          else { lo = lo_raw; hi = hi_raw; }
          lo = max(lo, x_first);
          hi = min(hi, x_last);
        }
        ctl->row_lo[s * 8 + tid] = lo;
        ctl->row_hi[s * 8 + tid] = hi;
      }
    }
  };

  // rotation angles of the slot this launch creates (boundary step): prepared in double by the last warp (ahead
  // of the wait when the launch may start early), kept in registers until the stages are free to hold them
  constexpr int kRopePerLane = D / 64;
  double rope_c[kRopePerLane], rope_s[kRopePerLane];

  // ---- Q^T fragments (B operand: 16 dims x 8 rows per step) straight from global memory into registers.
  // Thread (lane / 4, lane % 4) holds row lane / 4, dims 16 ks + 2 (lane % 4) + {0, 1} and + 8.
  const int gq = lane >> 2;
  const int q2 = (lane & 3) * 2;
  uint32_t qb[D / 16][2];
  int epoch_reg = 0;   // thread 0: this head's reduction epoch, kept in a register until the publication needs it
  auto wait_for_predecessor_and_load_q = [&]() {
    // a launch that was allowed to start early waits here for its predecessor, and lets its own successor start
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    MASW_STAMP(tr, 10);
    MASW_CLOCK(tr, 1);    // developer build, cycle stamps of thread 0: the wait has passed
    {
      const bool real = gq < n_rows;
      const int j = gq / p.G, g = gq % p.G;
      const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
          p.q + ((static_cast<size_t>(b) * p.n_q + (real ? j : 0)) * p.Hq + kvh * p.G + (real ? g : 0)) * D);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        qb[ks][0] = real ? __ldg(qrow + ks * 8 + (lane & 3)) : 0u;
        qb[ks][1] = real ? __ldg(qrow + ks * 8 + 4 + (lane & 3)) : 0u;
      }
    }
    if (tid == 0) epoch_reg = __ldcg(p.tickets + (b * p.Hkv + kvh) * (kMaxSplitsDev + 1));
  };

  // Without p.early everything follows the wait.  With it, the plan and the first ring of copies come first and
  // only q, the pending raw rows and the epoch are read behind the wait: the tiles are in shared memory by then.
  if (!p.early) wait_for_predecessor_and_load_q();
  plan_and_issue();
  if (warp == NW - 1 && p.h_g != nullptr) {
#pragma unroll
    for (int u = 0; u < kRopePerLane; ++u) {
      const int i = lane + 32 * u;
      sincos(static_cast<double>(p.slot_pos[b]) * pow(p.rope_base, -2.0 * i / D), &rope_s[u], &rope_c[u]);
    }
  }
  __syncthreads();   // the plan and the barriers are visible to every warp

  const int nseg = plan[0];
  const int tile_begin = plan[1];
  const int n_tiles = plan[2] - tile_begin;

  // ---- The register tile.  A CTA's share of a 32K-prefix memory is a little more than its seven stages
  // hold.  When the launch runs ahead of its predecessor (p.early) and has more than seven tiles, its first
  // tile is taken out of its stage before the wait: warp w keeps entries [8 w, 8 w + 8) of it as MMA fragments
  // (K rows as the A operand of S^T, V^T as the A operand of O^T: D / 4 registers), and the stage is handed
  // to tile 7 at once, so that eight tiles are on the chip when q arrives and nothing is fetched behind the wait.
  uint32_t kf[D / 16][2], vf[D / 16][2];
  bool reg_tile = false;
  int r_seg = 0, r_x0 = 0;
  if (p.early && n_tiles > NS) {
    while (r_seg + 1 < nseg && tile_begin >= plan[32 + r_seg + 1]) ++r_seg;
    const int i0 = (tile_begin - plan[32 + r_seg]) * TE;
    const int valid = min(TE, plan[8 + 4 * r_seg + 1] - i0);
    r_x0 = plan[8 + 4 * r_seg + 2] + i0;
    const int n_raw = p.n_q - p.last_row_is_slot;
    // never the tile that holds the pending raw tokens: their rows are patched in shared memory behind the wait
    const bool pending = p.k_raw != nullptr && plan[8 + 4 * r_seg + 3] != 1 &&
                         max(r_x0, plan[7]) < min(r_x0 + valid, plan[7] + n_raw);
    reg_tile = !pending;
    if (reg_tile) {
      bool okr = mbar_wait_bounded(&ctl->full_bar[0], 0, MASW_WAIT_LIMIT(p));
      okr = __all_sync(0xffffffffu, okr);
      if (!okr && lane == 0) {
        plan[3] = 1;
        if (p.status) atomicOr(p.status, MASW_STATUS_WAIT_TIMEOUT);
      }
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) { kf[ks][0] = kf[ks][1] = 0u; vf[ks][0] = vf[ks][1] = 0u; }
      if (okr && warp < TE / 8) {
        const uint32_t kb = smem_u32(pipe), vb = kb + C::kTileBytes;
        const int e = warp * 8 + (lane & 7);
        const int c1 = (lane >> 3) & 1;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const int cg = ks * 2 + c1;
          const uint32_t off = (cg >> 3) * C::kSubBytes + e * 128 + (((cg & 7) ^ (e & 7)) << 4);
          ldmatrix_x2(kf[ks][0], kf[ks][1], kb + off);          // (entry lane / 4; dims 16 ks + q2 + {0, 1}) and the same + 8
          ldmatrix_x2_trans(vf[ks][0], vf[ks][1], vb + off);    // (dim 16 ks + lane / 4; entries q2 + {0, 1}) and dim + 8
        }
        // entries of the tile beyond its segment hold foreign bytes: their V values must be zero
        const int e0 = warp * 8 + (lane & 3) * 2;
        const uint32_t keep = (e0 < valid ? 0x0000ffffu : 0u) | (e0 + 1 < valid ? 0xffff0000u : 0u);
#pragma unroll
        for (int md = 0; md < D / 16; ++md) { vf[md][0] &= keep; vf[md][1] &= keep; }
      }
      __syncthreads();   // every warp has its fragments: stage 0 is free for tile NS
      if (tid == 0) {
        const int it2 = tile_begin + NS;
        int sg = r_seg;
        while (sg + 1 < nseg && it2 >= plan[32 + sg + 1]) ++sg;
        const int row0 = plan[8 + 4 * sg] + (it2 - plan[32 + sg]) * TE;
        const uint64_t policy = l2_policy_evict_first();
        mbar_arrive_expect_tx(&ctl->full_bar[0], C::kStageBytes);
        st_release_shared(&ctl->armed[0], NS + 1);
#ifdef MASW_TRACE
        if (NS != p.drop_tile)
#endif
        {
#pragma unroll
          for (int sub = 0; sub < C::kSub; ++sub)
            tma_load_4d(pipe + sub * C::kSubBytes, &tmK, &ctl->full_bar[0], sub * 64, row0, kvh, b, policy);
#pragma unroll
          for (int sub = 0; sub < C::kSub; ++sub)
            tma_load_4d(pipe + C::kTileBytes + sub * C::kSubBytes, &tmV, &ctl->full_bar[0], sub * 64, row0, kvh, b, policy);
        }
      }
    }
  }

  if (p.early) {
    // L2 hints for what is read behind the wait (q, the pending raw rows, the slot projection's inputs).  A
    // prefetch reads no value, so a line the predecessor is still writing stays coherent; what it buys is an
    // L2 hit instead of a DRAM round trip on the path from the wait to the first scores.
    if (warp == 1) {
      const int lines = n_rows * (D / 64);
      if (lane < lines) {
        const int r = lane / (D / 64);
        prefetch_l2(p.q + ((static_cast<size_t>(b) * p.n_q + r / p.G) * p.Hq + kvh * p.G + r % p.G) * D + (lane % (D / 64)) * 64);
      }
    } else if (warp == 2 && p.k_raw != nullptr) {
      const int n_raw = p.n_q - p.last_row_is_slot;
      const int lines = n_raw * (D / 64);
      if (lane < 2 * lines) {
        const int l2 = lane % lines;
        const __nv_bfloat16* src = (lane < lines ? p.k_raw : p.v_raw) +
                                   ((static_cast<size_t>(b) * n_raw + l2 / (D / 64)) * p.Hkv + kvh) * D + (l2 % (D / 64)) * 64;
        prefetch_l2(src);
      }
    }
    if (p.h_g != nullptr) {
      const int k0 = static_cast<int>((static_cast<long long>(p.d_model) * split) / p.splits);
      const int k1 = static_cast<int>((static_cast<long long>(p.d_model) * (split + 1)) / p.splits);
      for (int k = k0 + tid; k < k1; k += C::kThreads) {
        const size_t off = static_cast<size_t>(k) * (p.Hkv * D) + kvh * D;
#pragma unroll
        for (int c = 0; c < D / 64; ++c) { prefetch_l2(p.Wk_g + off + c * 64); prefetch_l2(p.Wv_g + off + c * 64); }
      }
      if (tid == 0) prefetch_l2(p.h_g + static_cast<size_t>(b) * p.d_model + k0);
    }
    wait_for_predecessor_and_load_q();
  }

  // running state of a consumer thread: columns (query rows) q2, q2 + 1 of the S^T / O^T fragments
  float acc[D / 16][4];
  float m_run[2] = {kNegInf, kNegInf};
  float l_run[2] = {0.f, 0.f};
#pragma unroll
  for (int i = 0; i < D / 16; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }

  // ---- Geometry of a warp's next tile, prepared one tile ahead.  Fused append: the pending raw tokens
  // (positions t .. t + n_raw - 1) are not in memory yet; the warp that owns their tile overwrites their rows of
  // the landed tile in shared memory with the caller's K/V and also stores them to the arena for later steps
  // (nothing has to order that store against this launch's bulk copies).  The first chunks of those rows are
  // requested here, for a warp's first tile together with q, so their latency is not added to the tile's.
  constexpr int kPre = 2;
  const int t_b = plan[7];
  const int n_raw = p.n_q - p.last_row_is_slot;
  const int i_first = (reg_tile ? 1 : 0) + warp;
  int cur_seg = 0;
  int n_seg = 0, n_i0 = 0, n_x0 = 0, n_seglen = 0, n_pat_lo = 0, n_pat_per = 0;
  uint4 n_pre[kPre];
  auto raw_addr = [&](int idx, int pat_lo, int pat_per, int x0, int& which, int& r, int& cg) {
    which = idx / pat_per;
    const int rem = idx % pat_per;
    const int tok = pat_lo + rem / (D / 8);
    cg = rem % (D / 8);
    r = tok - x0;
    return reinterpret_cast<const uint4*>((which ? p.v_raw : p.k_raw) +
                                          ((static_cast<size_t>(b) * n_raw + (tok - t_b)) * p.Hkv + kvh) * D + cg * 8);
  };
  auto prepare = [&](int i) {
    n_pat_lo = 0; n_pat_per = 0;
    if (i >= n_tiles) return;
    const int it = tile_begin + i;
    while (cur_seg + 1 < nseg && it >= plan[32 + cur_seg + 1]) ++cur_seg;
    n_seg = cur_seg;
    n_i0 = (it - plan[32 + cur_seg]) * TE;
    n_seglen = plan[8 + 4 * cur_seg + 1];
    n_x0 = plan[8 + 4 * cur_seg + 2] + n_i0;
    if (p.k_raw != nullptr && plan[8 + 4 * cur_seg + 3] != 1) {
      const int lo = max(n_x0, t_b), hi = min(n_x0 + min(TE, n_seglen - n_i0), t_b + n_raw);   // inside this segment only
      if (lo < hi) {
        n_pat_lo = lo;
        n_pat_per = (hi - lo) * (D / 8);
#pragma unroll
        for (int u = 0; u < kPre; ++u) {
          const int idx = lane + 32 * u;
          if (idx < 2 * n_pat_per) {
            int which, r, cg;
            n_pre[u] = __ldg(raw_addr(idx, n_pat_lo, n_pat_per, n_x0, which, r, cg));
          }
        }
      }
    }
  };
  prepare(i_first);

  if (reg_tile) {
    // ---- this warp's eight entries of the register tile: S^T (rows 8..15 of the MMA are padding), softmax,
    //      O^T; they open the running softmax state
    float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int ks = 0; ks < D / 16; ++ks) {
      const uint32_t a[4] = {kf[ks][0], 0u, kf[ks][1], 0u};
      mma_bf16_16816(s4, a, qb[ks][0], qb[ks][1]);
    }
    const int x = r_x0 + warp * 8 + gq;
    const bool v0 = warp < TE / 8 && x >= ctl->row_lo[r_seg * 8 + q2] && x <= ctl->row_hi[r_seg * 8 + q2];
    const bool v1 = warp < TE / 8 && x >= ctl->row_lo[r_seg * 8 + q2 + 1] && x <= ctl->row_hi[r_seg * 8 + q2 + 1];
    const float s0 = v0 ? s4[0] * p.scale_log2e : kNegInf;
    const float s1 = v1 ? s4[1] * p.scale_log2e : kNegInf;
    float mx0 = s0, mx1 = s1;
#pragma unroll
    for (int o2 = 4; o2 <= 16; o2 <<= 1) {
      mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o2));
      mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o2));
    }
    m_run[0] = mx0; m_run[1] = mx1;
    const float p0 = fast_exp2(s0 - (mx0 == kNegInf ? 0.f : mx0)), p1 = fast_exp2(s1 - (mx1 == kNegInf ? 0.f : mx1));
    l_run[0] = p0; l_run[1] = p1;
    const uint32_t ha = pack_bf16x2(p0, p1);
    const float r0 = __uint_as_float(ha << 16), r1 = __uint_as_float(ha & 0xffff0000u);
    const uint32_t bh = movmatrix_trans(ha), bl = movmatrix_trans(pack_bf16x2(p0 - r0, p1 - r1));
#pragma unroll
    for (int md = 0; md < D / 16; ++md) {
      const uint32_t a[4] = {vf[md][0], vf[md][1], 0u, 0u};
      mma_bf16_16816(acc[md], a, bh, 0u);
      mma_bf16_16816(acc[md], a, bl, 0u);
    }
  }

#ifdef MASW_TRACE
  if (tr != nullptr && tid == 0) { if (qb[0][0] == 0xdeadbeefu) tr[15] = 1; tr[2] = clock64(); }   // q has arrived
#endif
  {
    // ================= the tiles in the stages =================
    const uint64_t policy = l2_policy_evict_first();
    int seg_bounds = -1;
    int lo0 = 1, hi0 = 0, lo1 = 1, hi1 = 0;   // visibility bounds of this thread's two columns in the current segment
    bool ok = true;

    for (int i = i_first; i < n_tiles; i += NW) {
      // the tile's geometry and the first chunks of its pending raw rows were prepared (and requested) ahead
      const int seg = n_seg, i0 = n_i0, x0 = n_x0, seg_len = n_seglen, pat_lo = n_pat_lo, pat_per = n_pat_per;
      uint4 pre[kPre];
#pragma unroll
      for (int u = 0; u < kPre; ++u) pre[u] = n_pre[u];
      if (seg != seg_bounds) {
        seg_bounds = seg;
        lo0 = ctl->row_lo[seg * 8 + q2]; hi0 = ctl->row_hi[seg * 8 + q2];
        lo1 = ctl->row_lo[seg * 8 + q2 + 1]; hi1 = ctl->row_hi[seg * 8 + q2 + 1];
      }
      const int stage = i % NS;
      const uint32_t parity = (i / NS) & 1;
      auto raw_src = [&](int idx, int& which, int& r, int& cg) { return raw_addr(idx, pat_lo, pat_per, x0, which, r, cg); };

      if (i >= NS) {   // a later round of this stage: wait until it has been re-armed for tile i
        int spins = 0;
        while (ld_acquire_shared(&ctl->armed[stage]) <= i && spins < MASW_WAIT_LIMIT(p)) { __nanosleep(40); ++spins; }
        ok = ld_acquire_shared(&ctl->armed[stage]) > i;
      }
      if (ok) ok = mbar_wait_bounded(&ctl->full_bar[stage], parity, MASW_WAIT_LIMIT(p));
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      MASW_CLOCK(tr, 3);    // warp 0's (last) tile has landed

      uint8_t* ksm = pipe + stage * C::kStageBytes;
      uint8_t* vsm = ksm + C::kTileBytes;
      const uint32_t ks_base = smem_u32(ksm);
      const uint32_t vs_base = smem_u32(vsm);

      if (pat_per > 0) {
        const int phys0 = plan[8 + 4 * seg] + i0;
        auto put = [&](int idx, uint4 val) {
          int which, r, cg;
          raw_src(idx, which, r, cg);
          uint8_t* tile = which ? vsm : ksm;
          *reinterpret_cast<uint4*>(tile + (cg >> 3) * C::kSubBytes + r * 128 + (((cg & 7) ^ (r & 7)) << 4)) = val;
          __nv_bfloat16* dst = (which ? p.v_base : p.k_base) + b * p.stride_b + kvh * p.stride_h +
                               static_cast<long long>(phys0 + r) * D + cg * 8;
          *reinterpret_cast<uint4*>(dst) = val;
        };
#pragma unroll
        for (int u = 0; u < kPre; ++u) {
          if (lane + 32 * u < 2 * pat_per) put(lane + 32 * u, pre[u]);
        }
        for (int idx = lane + 32 * kPre; idx < 2 * pat_per; idx += 32) {
          int which, r, cg;
          put(idx, __ldg(raw_src(idx, which, r, cg)));
        }
        fence_proxy_async();   // by every lane that wrote: the stage is handed back to the bulk copies later
        __syncwarp();
      }
      prepare(i + NW);   // the warp's next tile: geometry, and its pending rows (if any) requested now

      // entries of the tile beyond the segment hold foreign bytes: zero their V rows so that a zero
      // probability times a non-finite value cannot poison the accumulators
      const int valid = min(TE, seg_len - i0);
      if (valid < TE) {
        for (int idx = lane; idx < (TE - valid) * (D / 8); idx += 32) {
          const int r = valid + idx / (D / 8);
          const int cg = idx % (D / 8);
          *reinterpret_cast<uint4*>(vsm + (cg >> 3) * C::kSubBytes + r * 128 + ((cg & 7) << 4)) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async();
        __syncwarp();
      }

      // ---- S^T = K Q^T: 16 entries x 8 rows per MMA, A = K rows (ldmatrix), B = the Q^T fragments
      float st[TE / 16][4];
#ifdef MASW_TRACE
      if (p.debug_flags & 2) {
#pragma unroll
        for (int mt = 0; mt < TE / 16; ++mt) st[mt][0] = st[mt][1] = st[mt][2] = st[mt][3] = 0.f;
      } else
#endif
      {
        const int e_in = (lane & 7) + ((lane >> 3) & 1) * 8;   // row this lane addresses inside a 16-entry block
        const int c_hi = lane >> 4;                            // 0 / 1: first or second 8-dim chunk of the step
#pragma unroll
        for (int mt = 0; mt < TE / 16; ++mt) {
          st[mt][0] = st[mt][1] = st[mt][2] = st[mt][3] = 0.f;
          const int e = mt * 16 + e_in;
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            const int cg = ks * 2 + c_hi;
            uint32_t a[4];
            ldmatrix_x4(a[0], a[1], a[2], a[3], ks_base + (cg >> 3) * C::kSubBytes + e * 128 + (((cg & 7) ^ (e & 7)) << 4));
            mma_bf16_16816(st[mt], a, qb[ks][0], qb[ks][1]);
          }
        }
      }

      MASW_CLOCK(tr, 16);   // warp 0: scores of its (last) tile
      // ---- scale, mask, online softmax (exp2 domain).  st[mt][0..1]: entry 16 mt + gq, columns q2, q2 + 1;
      //      st[mt][2..3]: entry 16 mt + gq + 8
      const int x_last = x0 + TE - 1;
      const bool need_mask = (x0 < max(lo0, lo1)) || (x_last > min(hi0, hi1));
      float mx0 = kNegInf, mx1 = kNegInf;
#pragma unroll
      for (int mt = 0; mt < TE / 16; ++mt) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float v = st[mt][c] * p.scale_log2e;
          if (need_mask) {
            const int x = x0 + mt * 16 + gq + ((c & 2) ? 8 : 0);
            const bool vis = (c & 1) ? (x >= lo1 && x <= hi1) : (x >= lo0 && x <= hi0);
            v = vis ? v : kNegInf;
          }
          st[mt][c] = v;
        }
        mx0 = fmaxf(mx0, fmaxf(st[mt][0], st[mt][2]));
        mx1 = fmaxf(mx1, fmaxf(st[mt][1], st[mt][3]));
      }
#pragma unroll
      for (int o2 = 4; o2 <= 16; o2 <<= 1) {   // a column's entries live in the lanes that share lane % 4
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, o2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, o2));
      }
      const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
      const float mu0 = (mn0 == kNegInf) ? 0.f : mn0;
      const float mu1 = (mn1 == kNegInf) ? 0.f : mn1;
      if (__any_sync(0xffffffffu, mn0 != m_run[0] || mn1 != m_run[1])) {   // rescale only when some maximum moved
        const float c0 = fast_exp2(m_run[0] - mu0), c1 = fast_exp2(m_run[1] - mu1);
        m_run[0] = mn0; m_run[1] = mn1;
        l_run[0] *= c0; l_run[1] *= c1;
#pragma unroll
        for (int md = 0; md < D / 16; ++md) {
          acc[md][0] *= c0; acc[md][1] *= c1;
          acc[md][2] *= c0; acc[md][3] *= c1;
        }
      }

      // ---- P^T as the B operand of O^T += V^T P^T: the S^T fragment holds (entry = lane / 4, rows q2, q2 + 1);
      //      the operand wants (entries q2, q2 + 1; row = lane / 4): one 8 x 8 transpose per half block.
      //      p = p_hi + p_lo (two bf16 terms); the row sums use the unrounded values.
      uint32_t ph[TE / 16][2], pl[TE / 16][2];
#pragma unroll
      for (int mt = 0; mt < TE / 16; ++mt) {
        const float p0 = fast_exp2(st[mt][0] - mu0), p1 = fast_exp2(st[mt][1] - mu1);
        const float p2 = fast_exp2(st[mt][2] - mu0), p3 = fast_exp2(st[mt][3] - mu1);
        l_run[0] += p0 + p2;
        l_run[1] += p1 + p3;
        const uint32_t ha = pack_bf16x2(p0, p1), hb = pack_bf16x2(p2, p3);
        const float r0 = __uint_as_float(ha << 16), r1 = __uint_as_float(ha & 0xffff0000u);
        const float r2 = __uint_as_float(hb << 16), r3 = __uint_as_float(hb & 0xffff0000u);
        ph[mt][0] = movmatrix_trans(ha);
        ph[mt][1] = movmatrix_trans(hb);
        pl[mt][0] = movmatrix_trans(pack_bf16x2(p0 - r0, p1 - r1));
        pl[mt][1] = movmatrix_trans(pack_bf16x2(p2 - r2, p3 - r3));
      }

      MASW_CLOCK(tr, 17);   // ... probabilities in operand layout
      // ---- O^T += V^T P^T: A = V^T (16 dims x 16 entries) through transposing ldmatrix
#ifdef MASW_TRACE
      if (!(p.debug_flags & 2))
#endif
      {
        const int j = lane >> 3;
        const int e_in = (lane & 7) + (j >> 1) * 8;
#pragma unroll
        for (int mt = 0; mt < TE / 16; ++mt) {
          const int e = mt * 16 + e_in;
#pragma unroll
          for (int md = 0; md < D / 16; ++md) {
            const int cg = md * 2 + (j & 1);
            uint32_t a[4];
            ldmatrix_x4_trans(a[0], a[1], a[2], a[3], vs_base + (cg >> 3) * C::kSubBytes + e * 128 + (((cg & 7) ^ (e & 7)) << 4));
            mma_bf16_16816(acc[md], a, ph[mt][0], ph[mt][1]);
            mma_bf16_16816(acc[md], a, pl[mt][0], pl[mt][1]);
          }
        }
      }

      // ---- the stage is free: request the tile that follows in it (tile i + NS), if any
      __syncwarp();
      MASW_CLOCK(tr, 18);   // ... O^T updated
      if (lane == 0 && i + NS < n_tiles) {
        const int i2 = i + NS, it2 = tile_begin + i2;
        int sg = seg;
        while (sg + 1 < nseg && it2 >= plan[32 + sg + 1]) ++sg;
        const int row0 = plan[8 + 4 * sg] + (it2 - plan[32 + sg]) * TE;
        mbar_arrive_expect_tx(&ctl->full_bar[stage], C::kStageBytes);
        st_release_shared(&ctl->armed[stage], i2 + 1);   // armed for tile i2: its consumer may test the new phase
#ifdef MASW_TRACE
        if (i2 != p.drop_tile)
#endif
        {
#pragma unroll
          for (int sub = 0; sub < C::kSub; ++sub)
            tma_load_4d(ksm + sub * C::kSubBytes, &tmK, &ctl->full_bar[stage], sub * 64, row0, kvh, b, policy);
#pragma unroll
          for (int sub = 0; sub < C::kSub; ++sub)
            tma_load_4d(vsm + sub * C::kSubBytes, &tmV, &ctl->full_bar[stage], sub * 64, row0, kvh, b, policy);
        }
      }
    }
    MASW_CLOCK(tr, 19);     // warp 0 has left the tile loop
    if (!ok && lane == 0) {
      plan[3] = 1;
      if (p.status) atomicOr(p.status, MASW_STATUS_WAIT_TIMEOUT);
    }
    // row sums were kept per thread: finish them over the lanes that share the columns
#pragma unroll
    for (int o2 = 4; o2 <= 16; o2 <<= 1) {
      l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], o2);
      l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], o2);
    }
  }

  if (tid == 0) plan[6] = epoch_reg;
  __syncthreads();  // every tile consumed (or abandoned): the stages can be reused as scratch
  MASW_CLOCK(tr, 8);      // every warp's tiles are consumed
  if (plan[3] != 0) {
    // give-up path: a wait ran out.  Let this CTA's copies that are still in flight land (bounded) before
    // shared memory is reused or released; the outputs of this launch are not meaningful.
    if (tid < NS) {
      const int armed = ld_acquire_shared(&ctl->armed[tid]);
      if (armed > 0) mbar_wait_bounded(&ctl->full_bar[tid], ((armed - 1) / NS) & 1, MASW_WAIT_LIMIT(p));
    }
    __syncthreads();
  }

  // ---- per-warp partials -> shared memory: O^T fragment (dim 16 md + gq (+ 8), rows q2, q2 + 1)
  constexpr int kMS = C::kMergeStride;
  float* mo = reinterpret_cast<float*>(pipe + C::kMergeOff);   // [NW][8][kMS]
  float* mml = mo + NW * C::kRows * kMS;                       // [NW][8][2]
  double* rope_cs = reinterpret_cast<double*>(pipe + C::kRopeOff);
  {
    float* o0 = mo + (warp * C::kRows + q2) * kMS;
    float* o1 = o0 + kMS;
#pragma unroll
    for (int md = 0; md < D / 16; ++md) {
      o0[md * 16 + gq] = acc[md][0]; o1[md * 16 + gq] = acc[md][1];
      o0[md * 16 + gq + 8] = acc[md][2]; o1[md * 16 + gq + 8] = acc[md][3];
    }
    if (gq == 0) {
      mml[(warp * C::kRows + q2) * 2 + 0] = m_run[0]; mml[(warp * C::kRows + q2) * 2 + 1] = l_run[0];
      mml[(warp * C::kRows + q2 + 1) * 2 + 0] = m_run[1]; mml[(warp * C::kRows + q2 + 1) * 2 + 1] = l_run[1];
    }
  }
  if (warp == NW - 1 && p.h_g != nullptr) {
#pragma unroll
    for (int u = 0; u < kRopePerLane; ++u) {
      const int i = lane + 32 * u;
      rope_cs[2 * i] = rope_c[u]; rope_cs[2 * i + 1] = rope_s[u];
    }
  }
  __syncthreads();

  MASW_CLOCK(tr, 20);
  // ---- merge the warps' partials of each row into this split's partial and publish it as tagged records
  const int bh = b * p.Hkv + kvh;
  const int tag = plan[6] + 1;   // this launch's epoch tag
  {
    unsigned long long* po = p.part_o + (static_cast<size_t>(bh) * p.splits + split) * C::kRows * D;
    unsigned long long* pml = p.part_ml + (static_cast<size_t>(bh) * p.splits + split) * C::kRows * 2;
    for (int idx = tid; idx < n_rows * (D / 4); idx += C::kThreads) {
      const int r = idx / (D / 4);
      const int d4 = (idx % (D / 4)) * 4;
      float m = kNegInf;
#pragma unroll
      for (int e = 0; e < NW; ++e) m = fmaxf(m, mml[(e * C::kRows + r) * 2]);
      float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
      float l = 0.f;
#pragma unroll
      for (int e = 0; e < NW; ++e) {
        const float me = mml[(e * C::kRows + r) * 2];
        const float w = (me == kNegInf) ? 0.f : fast_exp2(me - m);
        const float4 v = *reinterpret_cast<const float4*>(mo + (e * C::kRows + r) * kMS + d4);
        o4.x += w * v.x; o4.y += w * v.y; o4.z += w * v.z; o4.w += w * v.w;
        l += w * mml[(e * C::kRows + r) * 2 + 1];
      }
      rec_store2(po + r * D + d4, o4.x, o4.y, tag);
      rec_store2(po + r * D + d4 + 2, o4.z, o4.w, tag);
      if (d4 == 0) rec_store2(pml + r * 2, m, l, tag);
    }
  }
  MASW_CLOCK(tr, 9);      // the partial is published

  // ---- fused slot materialisation, part 1 (boundary step): this CTA's slice of K_g = h_g W_K,g and
  //      V_g = h_g W_V,g for its KV head (rows [k0, k1) of the d_model contraction); the splits' partial sums
  //      are combined, rotated and used in split_reduce_and_store.  A thread owns eight columns (one 16-byte
  //      load per weight row) of every kRowLanes-th row.  It follows the attention partial so that the other
  //      splits can already fetch that while the weights stream.
  if (p.h_g != nullptr) {
    constexpr int kColThreads = D / 8;
    constexpr int kRowLanes = C::kThreads / kColThreads;
    constexpr int kChunk = 4;   // weight rows per thread and round trip
    const bool act = (p.active == nullptr) || (p.active[b] != 0);
    const int k0 = static_cast<int>((static_cast<long long>(p.d_model) * split) / p.splits);
    const int k1 = static_cast<int>((static_cast<long long>(p.d_model) * (split + 1)) / p.splits);
    __nv_bfloat16* hs = reinterpret_cast<__nv_bfloat16*>(pipe + C::kProjHsOff);     // [k1 - k0]
    float* red = reinterpret_cast<float*>(pipe + C::kProjRedOff);                    // [kRowLanes][2 * D]
    const int nk = min(k1 - k0, 8192);   // the staging area holds 16 KB of hidden state
    if (act) {
      for (int k = tid; k < nk; k += C::kThreads) hs[k] = p.h_g[static_cast<size_t>(b) * p.d_model + k0 + k];
    }
    __syncthreads();
    const int ct = tid % kColThreads, rl = tid / kColThreads;
    const int ncols = p.Hkv * D;
    float ak[8], av[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) { ak[c] = 0.f; av[c] = 0.f; }
    if (act && rl < kRowLanes) {
      for (int kb = k0 + rl; kb < k1; kb += kRowLanes * kChunk) {
        uint4 wk[kChunk], wv[kChunk];
#pragma unroll
        for (int u = 0; u < kChunk; ++u) {
          const int k = kb + u * kRowLanes;
          if (k < k1) {
            const size_t off = static_cast<size_t>(k) * ncols + kvh * D + ct * 8;
            wk[u] = __ldg(reinterpret_cast<const uint4*>(p.Wk_g + off));
            wv[u] = __ldg(reinterpret_cast<const uint4*>(p.Wv_g + off));
          }
        }
#pragma unroll
        for (int u = 0; u < kChunk; ++u) {
          const int k = kb + u * kRowLanes;
          if (k < k1) {
            const float x = (k - k0 < nk) ? __bfloat162float(hs[k - k0])
                                          : __bfloat162float(p.h_g[static_cast<size_t>(b) * p.d_model + k]);
            const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&wk[u]);
            const __nv_bfloat162* v2 = reinterpret_cast<const __nv_bfloat162*>(&wv[u]);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const float2 fk = __bfloat1622float2(k2[c]), fv = __bfloat1622float2(v2[c]);
              ak[2 * c] = fmaf(x, fk.x, ak[2 * c]); ak[2 * c + 1] = fmaf(x, fk.y, ak[2 * c + 1]);
              av[2 * c] = fmaf(x, fv.x, av[2 * c]); av[2 * c + 1] = fmaf(x, fv.y, av[2 * c + 1]);
            }
          }
        }
      }
    }
    if (rl < kRowLanes) {
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        red[rl * 2 * D + ct * 8 + c] = ak[c];
        red[rl * 2 * D + D + ct * 8 + c] = av[c];
      }
    }
    __syncthreads();
    unsigned long long* pslot = p.part_slot + (static_cast<size_t>(bh) * p.splits + split) * 2 * D;
    for (int c = tid; c < 2 * D; c += C::kThreads) {
      float a = 0.f;
      for (int l2 = 0; l2 < kRowLanes; ++l2) a += red[l2 * 2 * D + c];
      rec_store1(pslot + c, a, tag);
    }
  }

#ifdef MASW_TRACE
  if (tr && tid == 0) { tr[5] = 1; tr[6] = n_tiles; unsigned sm; asm("mov.u32 %0, %%smid;" : "=r"(sm)); tr[7] = sm; }
#endif
  // ---- cross-split reduction (see split_reduce_and_store)
#ifdef MASW_TRACE
  if (p.debug_flags & 1) return;
#endif
  split_reduce_and_store<D, C::kRows, C::kThreads>(p, b, kvh, split, n_rows, plan[6], reinterpret_cast<float*>(pipe + C::kReduceOff),
                                                   tid, p.h_g != nullptr ? rope_cs : nullptr
#ifdef MASW_TRACE
                                                   , tr
#endif
                                                   );
  MASW_CLOCK(tr, 13);
  MASW_STAMP(tr, 4);
}

}  // namespace masw
