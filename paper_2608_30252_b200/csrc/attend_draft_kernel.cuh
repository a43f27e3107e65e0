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
//    as hi + lo bf16 terms, which removes the bf16 rounding of the probabilities from the result.  With at most
//    four real rows (instance PACK) the two terms share one instruction: columns 4..7 of Q^T repeat rows 0..3,
//    their threads keep the remainders, and V^T P^T accumulates head and remainder side by side.
//  Instance SLOT carries the fused slot materialisation of the boundary step (h_g given); the plain decode launch
//  is compiled without it, so that its registers and its schedule do not pay for code it never runs.
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
  static constexpr int kReduceOff = 84 * 1024;                               // scratch of split_reduce_and_store
  static_assert(D == 64 || D == 128, "head_dim");
  static_assert(kMergeBytes <= kReduceOff, "merge scratch overlaps the reduction scratch");
  static_assert(kReduceOff + 9216 + 24 * D <= kPipeBytes, "reduction scratch must fit in the stages");
  static_assert(kThreads == 256, "draft_reduce_and_store is written for 256 threads");
  static_assert(kSmemBytes <= 113 * 1024, "two CTAs per SM");
};

struct DraftCtrl {
  uint64_t full_bar[8];
  int plan[40];        // [0] nseg, [1] tile_begin, [2] tile_end, [3] error flag, [6] reduction epoch, [7] committed tokens t,
                       // [8 + 4 s ..] phys, len, xbase, kind of segment s, [32 + s] first tile of segment s (s = 0..nseg)
  int row_lo[kMaxSeg * 8], row_hi[kMaxSeg * 8];
  int armed[8];        // per stage: 1 + the CTA-local index of the tile the stage was last armed (and requested) for
  float rope[128];     // boundary step: (cos, sin) of the new slot's D / 2 rotation angles (angles formed in double)
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


// Cross-split reduction of the draft launch: split_reduce_and_store's scheme (tagged 64-bit records, every CTA
// merges its slice of the (row, 4-column) items out of all splits' records in a fixed order) for eight rows and
// 256 threads, with the boundary step's slot work moved ahead of the rendezvous.  The splits' partial sums of
// K_g | V_g were published at the start of the launch, so they are here long before the attention partials:
// the CTAs that need the new slot (split 0 stores it; the owners of slot-row items attend to it) sum them in
// split order, rotate the key, round both to bf16 as stored and take the slot rows' scores against it while the
// other splits are still publishing; behind the rendezvous only the final combine is left.
// Must be called by all 256 threads; `scratch` is shared memory of at least 9 KB + 24 D bytes.
template <int D, bool SLOT>
__device__ __forceinline__ void draft_reduce_and_store(const AttendParams& p, int b, int kvh, int split, int n_rows, int epoch,
                                                       float* scratch, int tid, const float* rope_cs, long long* tr) {
  constexpr float kNegInf = -INFINITY;
  constexpr int NT = 256, KROWS = 8;
  constexpr int kGroups = 8, kSlots = NT / kGroups;   // thread groups per item, items per batch
  constexpr int kFetch = 3;   // splits whose records a group thread has in flight: 24 splits per round trip
  const int bh = b * p.Hkv + kvh;
  const int tag = epoch + 1;
  const unsigned long long* all_o = p.part_o + static_cast<size_t>(bh) * p.splits * KROWS * D;
  const unsigned long long* all_ml = p.part_ml + static_cast<size_t>(bh) * p.splits * KROWS * 2;
  const int splits = p.splits;
  const int n_items = n_rows * (D / 4);
  const int per = (n_items + splits - 1) / splits;
  const int i_begin = split * per;
  const int my_items = max(0, min(n_items, i_begin + per) - i_begin);
  float* gsm = scratch;                        // [kGroups][kSlots][6]: m, l, o4
  float* psum = gsm + kGroups * kSlots * 6;    // [NT / D][2 D] partial sums of K_g | V_g
  float* kg = psum + 2 * NT;                   // [D] key of the new slot (bf16 values); vg follows it
  float* vg = kg + D;
  float* sg = vg + D;                          // [G] scaled scores of the slot rows against it (log2 domain)
  bool timed_out = false;
  __syncthreads();   // the scratch is free

  // ---- boundary step: what the slot phase needs is requested now and used behind the rendezvous of the
  // attention partials (the splits published their sums of K_g | V_g at the start of the launch, so these
  // records have long arrived; the loads ride along with the wait for the other splits' partials)
  const int first_slot_item = (n_rows - p.G) * (D / 4);
  const bool slot_term = SLOT && p.h_g != nullptr && (p.active == nullptr || p.active[b] != 0) &&
                         (split == 0 || i_begin + my_items > first_slot_item);
  constexpr int kColGroups = NT / D;                        // thread (columns 2 c, 2 c + 1 of K | V, group): splits group, group + groups, ...
  constexpr int kBatch = (D == 64) ? 5 : 10;                // 16-byte record pairs in flight per thread: up to 20 splits in one round trip
  constexpr int kQPerLane = D / 32;
  const unsigned long long* ps = p.part_slot + static_cast<size_t>(bh) * splits * 2 * D;
  const int col = 2 * (tid % D), cgp = tid / D;
  const int warp = tid >> 5, lane = tid & 31;
  unsigned short qraw[kQPerLane];   // the slot rows' query values (warp g holds row g), converted when used
  MASW_CLOCK(tr, 26);     // developer build: the reduction starts
  if (slot_term) {
#pragma unroll
    for (int e = 0; e < kQPerLane; ++e) {
      qraw[e] = 0;
      if (warp < p.G)
        qraw[e] = __ldg(reinterpret_cast<const unsigned short*>(p.q) +
                        ((static_cast<size_t>(b) * p.n_q + (p.n_q - 1)) * p.Hq + kvh * p.G + warp) * D + lane + 32 * e);
    }
    // the splits' sums of this thread's column, in split order; the total goes to shared memory at once, so that
    // nothing is held in registers while the attention partials are awaited
    float sum = 0.f, sum_b = 0.f;
    for (int sp0 = cgp; sp0 < splits; sp0 += kColGroups * kBatch) {
      float sv[kBatch], sw[kBatch];
      bool sok[kBatch];
      bool all_ok = true;
#pragma unroll
      for (int e = 0; e < kBatch; ++e) {
        sv[e] = 0.f; sw[e] = 0.f; sok[e] = true;
        const int sp = sp0 + e * kColGroups;
        if (sp < splits) {
          const Rec2 r = rec_load2(ps + static_cast<size_t>(sp) * 2 * D + col, tag);
          sv[e] = r.a; sw[e] = r.b; sok[e] = r.ok; all_ok &= r.ok;
        }
      }
#ifdef MASW_TRACE
      if (tr != nullptr && tid == 0) { tr[29] = clock64(); tr[30] = all_ok ? 1 : 2; }   // first answers are in; were they all there?
#endif
      for (int it = 0; !all_ok && it < MASW_WAIT_LIMIT(p); ++it) {   // a split that has not published yet
        __nanosleep(20);
        all_ok = true;
#pragma unroll
        for (int e = 0; e < kBatch; ++e) {
          if (!sok[e]) {
            const Rec2 r = rec_load2(ps + static_cast<size_t>(sp0 + e * kColGroups) * 2 * D + col, tag);
            sv[e] = r.a; sw[e] = r.b; sok[e] = r.ok; all_ok &= r.ok;
          }
        }
      }
      timed_out |= !all_ok;
#pragma unroll
      for (int e = 0; e < kBatch; ++e) { sum += sv[e]; sum_b += sw[e]; }
    }
    psum[cgp * 2 * D + col] = sum;
    psum[cgp * 2 * D + col + 1] = sum_b;
    MASW_CLOCK(tr, 25);   // developer build: this thread's slot records are summed
  }
  // The rest of the slot phase; called by the whole CTA once the first batch of items has its records (a
  // __syncthreads() lies between the sums above and this).
  auto slot_phase = [&]() {
    // unit u < D / 2: key columns (u, u + D / 2), rotated together; unit D / 2 + j: value columns (2 j, 2 j + 1)
    if (tid < D) {
      const int u = tid;
      const bool is_k = u < D / 2;
      const int c0 = is_k ? u : D + 2 * (u - D / 2);
      const int c1 = is_k ? u + D / 2 : c0 + 1;
      float sum0 = 0.f, sum1 = 0.f;
#pragma unroll
      for (int g2 = 0; g2 < kColGroups; ++g2) { sum0 += psum[g2 * 2 * D + c0]; sum1 += psum[g2 * 2 * D + c1]; }
      if (is_k) {
        const float cs = rope_cs[2 * u], sn = rope_cs[2 * u + 1];
        const float x1 = sum0, x2 = sum1;
        sum0 = fmaf(x1, cs, -x2 * sn);
        sum1 = fmaf(x2, cs, x1 * sn);
      }
      kg[c0] = __bfloat162float(__float2bfloat16_rn(sum0));   // kg | vg are contiguous; values as stored
      kg[c1] = __bfloat162float(__float2bfloat16_rn(sum1));
    }
    __syncthreads();
    MASW_CLOCK(tr, 27);   // ... the new slot's key and value are final
    if (warp < p.G) {   // scores of the G slot rows: one warp per row
      float dot = 0.f;
#pragma unroll
      for (int e = 0; e < kQPerLane; ++e)
        dot = fmaf(__uint_as_float(static_cast<unsigned>(qraw[e]) << 16), kg[lane + 32 * e], dot);
      for (int o2 = 16; o2 > 0; o2 >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o2);
      if (lane == 0) sg[warp] = dot * p.scale_log2e;
    }
    if (split == 0) {
      const int m_slot = p.n_slots[b] + p.dm;
      if (m_slot < p.max_slots) {
        for (int c = tid; c < 2 * D; c += NT) {
          __nv_bfloat16* dst = (c < D ? p.k_base : p.v_base) + b * p.stride_b + kvh * p.stride_h +
                               static_cast<long long>(p.S + m_slot) * D + (c % D);
          *dst = __float2bfloat16_rn(kg[c]);
        }
      } else if (tid == 0 && p.status) {
        atomicOr(p.status, MASW_STATUS_SLOT_OVERFLOW);
      }
    }
    __syncthreads();
    MASW_CLOCK(tr, 28);   // ... the slot phase is over
  };

  for (int base = 0; base < my_items; base += kSlots) {
    const int li = base + tid / kGroups;      // local item
    const int grp = tid % kGroups;
    const bool live = li < my_items;
    const int idx = i_begin + (live ? li : 0);
    const int r = idx / (D / 4);
    const int d4 = (idx % (D / 4)) * 4;
    float m_run2 = kNegInf, l_run2 = 0.f;
    float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
    // everything the final combine needs besides the partials is worked out before the records are awaited
    const int j = r / p.G, g = r % p.G;
    const size_t row_off = (static_cast<size_t>(b) * p.n_q + j) * p.Hq + kvh * p.G + g;
    float* const out_o = p.o + row_off * D + d4;
    __nv_bfloat16* const out_bf16 = p.o_bf16 ? p.o_bf16 + row_off * D + d4 : nullptr;
    float* const out_lse = (d4 == 0 && p.lse) ? p.lse + row_off : nullptr;
    const bool with_slot = slot_term && idx >= first_slot_item;
    const float* const my_gsm = gsm + (tid / kGroups) * 6;
    if (live) {
      for (int sp0 = grp; sp0 < splits; sp0 += kGroups * kFetch) {
        float2 ml[kFetch];
        float4 v[kFetch];
        bool okv[kFetch];
        bool all_ok = true;
#pragma unroll
        for (int u = 0; u < kFetch; ++u) {
          okv[u] = true;
          const int sp = sp0 + u * kGroups;
          if (sp < splits) {
            rec_fetch_item(all_ml + (sp * KROWS + r) * 2, all_o + (static_cast<size_t>(sp) * KROWS + r) * D + d4, tag, ml[u],
                           v[u], okv[u]);
            all_ok &= okv[u];
          }
        }
        for (int it = 0; !all_ok && it < MASW_WAIT_LIMIT(p); ++it) {   // a split that has not published yet
          __nanosleep(20);
          all_ok = true;
#pragma unroll
          for (int u = 0; u < kFetch; ++u) {
            if (!okv[u]) {
              const int sp = sp0 + u * kGroups;
              rec_fetch_item(all_ml + (sp * KROWS + r) * 2, all_o + (static_cast<size_t>(sp) * KROWS + r) * D + d4, tag,
                             ml[u], v[u], okv[u]);
              all_ok &= okv[u];
            }
          }
        }
        timed_out |= !all_ok;
        MASW_CLOCK(tr, 11);   // developer build: thread 0 holds every split's record of its first item
        float mb = m_run2;
#pragma unroll
        for (int u = 0; u < kFetch; ++u) if (sp0 + u * kGroups < splits) mb = fmaxf(mb, ml[u].x);
        const float mu = (mb == kNegInf) ? 0.f : mb;
        const float c = fast_exp2(m_run2 - mu);
        o4.x *= c; o4.y *= c; o4.z *= c; o4.w *= c;
        l_run2 *= c;
        m_run2 = mb;
#pragma unroll
        for (int u = 0; u < kFetch; ++u) {
          if (sp0 + u * kGroups < splits) {
            const float w = fast_exp2(ml[u].x - mu);   // exp2(-inf) = 0 for an empty split
            o4.x += w * v[u].x; o4.y += w * v[u].y; o4.z += w * v[u].z; o4.w += w * v[u].w;
            l_run2 += w * ml[u].y;
          }
        }
      }
      float* dst = gsm + (grp * kSlots + tid / kGroups) * 6;
      dst[0] = m_run2; dst[1] = l_run2; dst[2] = o4.x; dst[3] = o4.y; dst[4] = o4.z; dst[5] = o4.w;
    }
    __syncthreads();
    MASW_CLOCK(tr, 12);     // developer build: every item of this CTA has all its records
    if (base == 0 && slot_term) slot_phase();
    const float s_new = with_slot ? sg[g] : 0.f;
    const float4 v_new = with_slot ? make_float4(vg[d4], vg[d4 + 1], vg[d4 + 2], vg[d4 + 3]) : make_float4(0.f, 0.f, 0.f, 0.f);
    if (live && grp == 0) {
      // the groups' partials (m, l | o.x, o.y | o.z, o.w), merged in group order
      float m = kNegInf;
#pragma unroll
      for (int g2 = 0; g2 < kGroups; ++g2) m = fmaxf(m, my_gsm[g2 * kSlots * 6]);
      if (with_slot) m = fmaxf(m, s_new);
      float l = 0.f;
      float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int g2 = 0; g2 < kGroups; ++g2) {
        const float2 ml2 = *reinterpret_cast<const float2*>(my_gsm + g2 * kSlots * 6);
        const float2 oa = *reinterpret_cast<const float2*>(my_gsm + g2 * kSlots * 6 + 2);
        const float2 ob = *reinterpret_cast<const float2*>(my_gsm + g2 * kSlots * 6 + 4);
        const float w = (ml2.x == kNegInf) ? 0.f : fast_exp2(ml2.x - m);
        l += w * ml2.y;
        o.x += w * oa.x; o.y += w * oa.y; o.z += w * ob.x; o.w += w * ob.y;
      }
      if (with_slot) {
        const float w_new = fast_exp2(s_new - m);
        l += w_new;
        o.x += w_new * v_new.x; o.y += w_new * v_new.y; o.z += w_new * v_new.z; o.w += w_new * v_new.w;
      }
      MASW_CLOCK(tr, 21);     // developer build: combined, before the stores
      const float inv = (l > 0.f) ? __frcp_rn(l) : 0.f;
      o.x *= inv; o.y *= inv; o.z *= inv; o.w *= inv;
      *reinterpret_cast<float4*>(out_o) = o;
      if (out_bf16) *reinterpret_cast<uint2*>(out_bf16) = make_uint2(pack_bf16x2(o.x, o.y), pack_bf16x2(o.z, o.w));
      if (out_lse) *out_lse = (l > 0.f) ? (m + __log2f(l)) * 0.6931471805599453f : kNegInf;
    }
    MASW_CLOCK(tr, 22);     // developer build: this CTA's outputs are stored
    if (base + kSlots < my_items) __syncthreads();   // the group partials are overwritten by the next batch of items
  }
  if (timed_out && p.status) atomicOr(p.status, MASW_STATUS_WAIT_TIMEOUT);
  // every split has published records tagged with this launch's epoch, so all of them have read the old one
  if (split == 0 && tid == 0) p.tickets[bh * (kMaxSplitsDev + 1)] = tag;
}

template <int D, bool PACK, bool SLOT>
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

#ifdef MASW_TRACE
  if (p.debug_flags & 8) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // timing experiment: successor released at once
#endif
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
      // split s takes tiles [ceil(acc s / splits), ceil(acc (s + 1) / splits)): where the tiles do not divide evenly
      // the LAST split, which also patches the pending raw rows into its last tile, is among the short ones
      plan[1] = static_cast<int>((static_cast<long long>(acc) * split + p.splits - 1) / p.splits);
      plan[2] = static_cast<int>((static_cast<long long>(acc) * (split + 1) + p.splits - 1) / p.splits);
      plan[3] = 0;
      plan[7] = t_b;
    }
    if (is_producer) {
      int first[kMaxSeg + 1];
      int acc = 0;
      for (int s = 0; s < nseg; ++s) { first[s] = acc; acc += (seg[s].len + TE - 1) / TE; }
      first[nseg] = acc;
      const int tb = static_cast<int>((static_cast<long long>(acc) * split + p.splits - 1) / p.splits);
      const int te = static_cast<int>((static_cast<long long>(acc) * (split + 1) + p.splits - 1) / p.splits);
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

  // rotation angles of the slot this launch creates (boundary step): formed in double by the last warp (ahead of
  // the wait when the launch may start early); their cosine and sine are kept as fp32 in the control block
  // (the rotated key is rounded to bf16, so fp32 factors lose nothing)
  constexpr int kRopePerLane = D / 64;

  // ---- Q^T fragments (B operand: 16 dims x 8 rows per step) straight from global memory into registers.
  // Thread (lane / 4, lane % 4) holds row lane / 4, dims 16 ks + 2 (lane % 4) + {0, 1} and + 8.
  const int gq = lane >> 2;
  const int q2 = (lane & 3) * 2;
  // PACK (at most four real rows): MMA columns 4..7 repeat rows 0..3, so the scores come out twice; the threads
  // of columns 0..3 carry the bf16 head of each probability and those of columns 4..7 its bf16 remainder, and ONE
  // V^T P^T instruction per block accumulates both terms (in columns c and c + 4, added when the warps merge)
  const int gr = PACK ? (gq & 3) : gq;      // query row of this thread's Q^T column
  const int qc = PACK ? (q2 & 3) : q2;      // query row of this thread's first S^T / O^T column
  const bool lo_term = PACK && (lane & 2);  // this thread's columns carry the remainders
  uint32_t qb[D / 16][2];
  int epoch_reg = 0;   // this head's reduction epoch (every thread loads it: one broadcast transaction per warp)
  auto wait_for_predecessor_and_load_q = [&]() {
    // a launch that was allowed to start early waits here for its predecessor, and lets its own successor start
    MASW_CLOCK(tr, 14);   // developer build: thread 0 reaches the wait (its work ahead of the predecessor is done)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    MASW_STAMP(tr, 10);
    MASW_CLOCK(tr, 1);    // developer build, cycle stamps of thread 0: the wait has passed
    {
      const bool real = gr < n_rows;
      const int j = gr / p.G, g = gr % p.G;
      const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
          p.q + ((static_cast<size_t>(b) * p.n_q + (real ? j : 0)) * p.Hq + kvh * p.G + (real ? g : 0)) * D);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        qb[ks][0] = real ? __ldg(qrow + ks * 8 + (lane & 3)) : 0u;
        qb[ks][1] = real ? __ldg(qrow + ks * 8 + 4 + (lane & 3)) : 0u;
      }
    }
    epoch_reg = __ldcg(p.tickets + (b * p.Hkv + kvh) * (kMaxSplitsDev + 1));
  };

  // ---- fused slot materialisation, part 1 (boundary step): this CTA's slice of K_g = h_g W_K,g and V_g = h_g W_V,g
  //      for its KV head (rows [pk0, pk1) of the d_model contraction), in registers only: warp w owns 2 D / 8 of
  //      the head's 2 D output columns (K | V), a lane one 16-byte chunk of every (32 / chunks)-th weight row.
  //      The mirrored projections are parameters, which no launch of a decoding step writes: with p.early their
  //      rows are requested ahead of the wait and only h_g is read behind it.
  constexpr int kProjColsPerWarp = 2 * D / NW;        // 16 or 32
  constexpr int kProjChunks = kProjColsPerWarp / 8;   // 16-byte chunks of a row this warp reads: 2 or 4
  constexpr int kProjRowLanes = 32 / kProjChunks;
  constexpr int kProjInFlight = 8;                    // weight rows per lane and round trip
  const bool proj_on = SLOT && p.h_g != nullptr && (p.active == nullptr || p.active[b] != 0);
  const int prl = lane / kProjChunks;
  const int pcol = warp * kProjColsPerWarp + (lane % kProjChunks) * 8;   // first of this lane's eight columns in K | V
  const int pk0 = static_cast<int>((static_cast<long long>(p.d_model) * split) / p.splits);
  const int pk1 = static_cast<int>((static_cast<long long>(p.d_model) * (split + 1)) / p.splits);
  uint4 pw[kProjInFlight];
  auto proj_load_weights = [&](int kb) {
    const __nv_bfloat16* W = (pcol < D ? p.Wk_g : p.Wv_g) + kvh * D + (pcol < D ? pcol : pcol - D);
    const int ncols = p.Hkv * D;
#pragma unroll
    for (int u = 0; u < kProjInFlight; ++u) {
      const int k = kb + u * kProjRowLanes;
      pw[u] = make_uint4(0, 0, 0, 0);
      if (k < pk1) pw[u] = __ldg(reinterpret_cast<const uint4*>(W + static_cast<size_t>(k) * ncols));
    }
  };

  // Without p.early everything follows the wait.  With it, the plan and the first ring of copies come first and
  // only q, the pending raw rows and the epoch are read behind the wait: the tiles are in shared memory by then.
  if (!p.early) {
    // The launch in front may still be writing the counters (a counter update, a rollback) or the arena, so
    // nothing is READ for use ahead of the wait.  But this CTA's tiles can be asked into L2 from a guess: the
    // counters as they stand now (one step old at worst) name almost the same entries, a prefetch returns no
    // data, and a wrong guess costs nothing but the hint.  The real plan follows behind the wait.  (Only where the
    // launch's KV is small beside L2: at batch 16 the predecessor streams twice the L2's size past the hinted
    // lines before they are used, and the hint then cost 6 % of the launch.)
    if (is_producer && p.guess_hint) {
      Segment seg[kMaxSeg];
      int t_g, m_g;
      const int nseg_g = build_segments<true>(p, b, seg, t_g, m_g);
      int first[kMaxSeg + 1];
      int acc = 0;
      for (int s = 0; s < nseg_g; ++s) { first[s] = acc; acc += (seg[s].len + TE - 1) / TE; }
      first[nseg_g] = acc;
      const int tb = static_cast<int>((static_cast<long long>(acc) * split + p.splits - 1) / p.splits);
      const int te = static_cast<int>((static_cast<long long>(acc) * (split + 1) + p.splits - 1) / p.splits);
      int sg = 0;
      for (int it = tb; it < min(te, tb + NS + 1); ++it) {
        while (sg + 1 < nseg_g && it >= first[sg + 1]) ++sg;
        const int row0 = seg[sg].phys + (it - first[sg]) * TE;
#pragma unroll
        for (int sub = 0; sub < C::kSub; ++sub) {
          tma_prefetch_4d(&tmK, sub * 64, row0, kvh, b);
          tma_prefetch_4d(&tmV, sub * 64, row0, kvh, b);
        }
      }
    }
    wait_for_predecessor_and_load_q();
    if (proj_on) proj_load_weights(pk0 + prl);
  }
  plan_and_issue();
  if (SLOT && warp == NW - 1 && p.h_g != nullptr) {
#pragma unroll
    for (int u = 0; u < kRopePerLane; ++u) {
      const int i = lane + 32 * u;
      double sn, cs;
      sincos(static_cast<double>(p.slot_pos[b]) * pow(p.rope_base, -2.0 * i / D), &sn, &cs);
      ctl->rope[2 * i] = static_cast<float>(cs);
      ctl->rope[2 * i + 1] = static_cast<float>(sn);
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
    if (proj_on) {
      // the slot token's hidden state arrives with q; the weight rows are requested here, ahead of the wait
      for (int k = pk0 + tid * 64; k < pk1; k += C::kThreads * 64) prefetch_l2(p.h_g + static_cast<size_t>(b) * p.d_model + k);
      proj_load_weights(pk0 + prl);
    }
    wait_for_predecessor_and_load_q();
  }

  // running state of a consumer thread: columns (query rows) q2, q2 + 1 of the S^T / O^T fragments
  float acc[D / 16][4];
  float m_run[2] = {kNegInf, kNegInf};
  float l_run[2] = {0.f, 0.f};
#pragma unroll
  for (int i = 0; i < D / 16; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }

  // ---- fused slot materialisation, part 1, the arithmetic (the weight rows were requested above): h_g arrives
  //      with q, the row lanes are summed with shuffles, and the warp publishes its columns of the split's
  //      partial sums at once.  By the time the attention partials meet, these records have long arrived; they
  //      are combined, rotated and used in draft_reduce_and_store.
  if (proj_on) {
    const __nv_bfloat16* h = p.h_g + static_cast<size_t>(b) * p.d_model;
    float a8[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) a8[c] = 0.f;
    for (int kb = pk0 + prl; kb < pk1; kb += kProjRowLanes * kProjInFlight) {
      float x[kProjInFlight];
#pragma unroll
      for (int u = 0; u < kProjInFlight; ++u) {
        const int k = kb + u * kProjRowLanes;
        x[u] = (k < pk1) ? __bfloat162float(h[k]) : 0.f;
      }
      if (kb != pk0 + prl) proj_load_weights(kb);   // a long slice: the later batches are requested here
      MASW_CLOCK(tr, 23);   // developer build: the projection's inputs are requested
#pragma unroll
      for (int u = 0; u < kProjInFlight; ++u) {
        const __nv_bfloat162* w2 = reinterpret_cast<const __nv_bfloat162*>(&pw[u]);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const float2 f = __bfloat1622float2(w2[c]);
          a8[2 * c] = fmaf(x[u], f.x, a8[2 * c]);
          a8[2 * c + 1] = fmaf(x[u], f.y, a8[2 * c + 1]);
        }
      }
    }
#pragma unroll
    for (int off = kProjChunks; off < 32; off <<= 1) {
#pragma unroll
      for (int c = 0; c < 8; ++c) a8[c] += __shfl_xor_sync(0xffffffffu, a8[c], off);
    }
    MASW_CLOCK(tr, 24);     // ... its sums are complete
    if (prl == 0) {
      unsigned long long* pslot = p.part_slot + (static_cast<size_t>(b * p.Hkv + kvh) * p.splits + split) * 2 * D + pcol;
#pragma unroll
      for (int c = 0; c < 8; c += 2) rec_store2(pslot + c, a8[c], a8[c + 1], epoch_reg + 1);
    }
  }

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
    const bool v0 = warp < TE / 8 && x >= ctl->row_lo[r_seg * 8 + qc] && x <= ctl->row_hi[r_seg * 8 + qc];
    const bool v1 = warp < TE / 8 && x >= ctl->row_lo[r_seg * 8 + qc + 1] && x <= ctl->row_hi[r_seg * 8 + qc + 1];
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
    if constexpr (PACK) {
      const uint32_t bx = movmatrix_trans(lo_term ? pack_bf16x2(p0 - r0, p1 - r1) : ha);
#pragma unroll
      for (int md = 0; md < D / 16; ++md) {
        const uint32_t a[4] = {vf[md][0], vf[md][1], 0u, 0u};
        mma_bf16_16816(acc[md], a, bx, 0u);
      }
    } else {
      const uint32_t bh = movmatrix_trans(ha), bl = movmatrix_trans(pack_bf16x2(p0 - r0, p1 - r1));
#pragma unroll
      for (int md = 0; md < D / 16; ++md) {
        const uint32_t a[4] = {vf[md][0], vf[md][1], 0u, 0u};
        mma_bf16_16816(acc[md], a, bh, 0u);
        mma_bf16_16816(acc[md], a, bl, 0u);
      }
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
        lo0 = ctl->row_lo[seg * 8 + qc]; hi0 = ctl->row_hi[seg * 8 + qc];
        lo1 = ctl->row_lo[seg * 8 + qc + 1]; hi1 = ctl->row_hi[seg * 8 + qc + 1];
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
      uint32_t ph[TE / 16][2], pl[PACK ? 1 : TE / 16][2];   // PACK: ph holds head | remainder columns, pl is unused
#pragma unroll
      for (int mt = 0; mt < TE / 16; ++mt) {
        const float p0 = fast_exp2(st[mt][0] - mu0), p1 = fast_exp2(st[mt][1] - mu1);
        const float p2 = fast_exp2(st[mt][2] - mu0), p3 = fast_exp2(st[mt][3] - mu1);
        l_run[0] += p0 + p2;
        l_run[1] += p1 + p3;
        const uint32_t ha = pack_bf16x2(p0, p1), hb = pack_bf16x2(p2, p3);
        const float r0 = __uint_as_float(ha << 16), r1 = __uint_as_float(ha & 0xffff0000u);
        const float r2 = __uint_as_float(hb << 16), r3 = __uint_as_float(hb & 0xffff0000u);
        if constexpr (PACK) {
          ph[mt][0] = movmatrix_trans(lo_term ? pack_bf16x2(p0 - r0, p1 - r1) : ha);
          ph[mt][1] = movmatrix_trans(lo_term ? pack_bf16x2(p2 - r2, p3 - r3) : hb);
        } else {
          ph[mt][0] = movmatrix_trans(ha);
          ph[mt][1] = movmatrix_trans(hb);
          pl[mt][0] = movmatrix_trans(pack_bf16x2(p0 - r0, p1 - r1));
          pl[mt][1] = movmatrix_trans(pack_bf16x2(p2 - r2, p3 - r3));
        }
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
            if constexpr (!PACK) mma_bf16_16816(acc[md], a, pl[mt][0], pl[mt][1]);
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
  const float* rope_cs = ctl->rope;
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
        float4 v = *reinterpret_cast<const float4*>(mo + (e * C::kRows + r) * kMS + d4);
        if constexpr (PACK) {   // columns r + 4 accumulated the remainder terms of row r
          const float4 v2 = *reinterpret_cast<const float4*>(mo + (e * C::kRows + r + 4) * kMS + d4);
          v.x += v2.x; v.y += v2.y; v.z += v2.z; v.w += v2.w;
        }
        o4.x += w * v.x; o4.y += w * v.y; o4.z += w * v.z; o4.w += w * v.w;
        l += w * mml[(e * C::kRows + r) * 2 + 1];
      }
      rec_store2(po + r * D + d4, o4.x, o4.y, tag);
      rec_store2(po + r * D + d4 + 2, o4.z, o4.w, tag);
      if (d4 == 0) rec_store2(pml + r * 2, m, l, tag);
    }
  }
  MASW_CLOCK(tr, 9);      // the partial is published

#ifdef MASW_TRACE
  if (tr && tid == 0) { tr[5] = 1; tr[6] = n_tiles; unsigned sm; asm("mov.u32 %0, %%smid;" : "=r"(sm)); tr[7] = sm; }
#endif
  // ---- cross-split reduction
#ifdef MASW_TRACE
  if (p.debug_flags & 1) return;
#else
  long long* tr = nullptr;
#endif
  draft_reduce_and_store<D, SLOT>(p, b, kvh, split, n_rows, plan[6], reinterpret_cast<float*>(pipe + C::kReduceOff), tid, rope_cs, tr);
  MASW_CLOCK(tr, 13);
  MASW_STAMP(tr, 4);
}

}  // namespace masw
