// Split-K flash-decode attention kernel shared by draft_attend and verify_attend.
//
// One CTA owns one (sequence, KV head, split): a contiguous run of KV tiles out of the entries that
// are visible to at least one query row.  A producer warp streams K and V tiles [TE entries x D] from
// HBM into a ring of 128B-swizzled shared-memory stages with TMA bulk tensor copies (completion on
// mbarriers with transaction counts).  MT*EW consumer warps each own one 16-row block of the
// (tokens x group heads) query tile and every EW-th KV tile; they compute S = Q K^T and O += P V on
// the tensor cores (bf16 inputs, fp32 accumulate) with an online softmax in the exp2 domain.
// The EW partial results per row block are merged through shared memory and written as a split
// partial to global scratch; the splits of a (sequence, KV head) then meet on an arrival counter
// (cooperative launch, bounded wait) and each merges a slice of the rows in split order.
// (Running an L2 prefetch ahead of the ring was measured twice and dropped: as bulk-tensor prefetches
// it costs the per-SM TMA unit, which bounds the streaming rate with 128-byte rows, a second pass per
// box; as per-line prefetch instructions from the producer warp it slowed the stream by 40 %.)
#pragma once

#include "common.cuh"

namespace masw {

constexpr int kMaxSeg = 4;
constexpr int kMaxSplitsDev = 64;   // upper bound on splits per (sequence, KV head); the host clamps to it

struct AttendParams {
  const __nv_bfloat16* q;  // [B][n_q][Hq][D]
  // fused raw-token append (draft only, null otherwise): the pending tokens' K/V [B][n_raw][Hkv][D] and the
  // K / V tensors of the layer they are appended to
  const __nv_bfloat16* k_raw;
  const __nv_bfloat16* v_raw;
  __nv_bfloat16* k_base;
  __nv_bfloat16* v_base;
  long long stride_b, stride_h;  // elements between sequences / KV heads of k_base, v_base (entries are D apart)
  // fused slot materialisation (draft boundary step only, null otherwise): the slot token's hidden state
  // [B][d_model], the layer's mirrored projections [d_model][Hkv*D], the slot's RoPE position and the
  // per-sequence mask; part_slot [B*Hkv][splits][2*D] receives the k-split partial sums of K_g | V_g
  const __nv_bfloat16* h_g;
  const __nv_bfloat16* Wk_g;
  const __nv_bfloat16* Wv_g;
  const int* slot_pos;
  const unsigned char* active;
  unsigned long long* part_slot;
  int d_model;
  double rope_base;
  float* o;                // [B][n_q][Hq][D]
  float* lse;              // [B][n_q][Hq] or null
  __nv_bfloat16* o_bf16;   // or null
  unsigned long long* part_o;   // [B*Hkv][splits][rows][D] tagged records (see rec_* below)
  unsigned long long* part_ml;  // [B*Hkv][splits][rows][2]: m, l
  int* tickets;            // [B*Hkv][1 + kMaxSplitsDev]: word 0 = reduction epoch of this (sequence, KV head)
  int* status;             // device status word (may be null)
  const int* t;            // draft: committed raw tokens per sequence
  const int* n_slots;      // draft: committed slots per sequence
  const int* kv_len;       // verify: entries in use per sequence (null selects the draft plan)
  int n_q, last_row_is_slot;
  int G, Hq, Hkv;
  int S, W, ring_cap, max_slots;
  int capacity;            // entries per (sequence, head) in the tensor map (paged: logical entries per sequence)
  const int* page_table;   // paged verifier cache: [B][max_pages] physical page of each 128-entry logical page, else null
  const float* k_scale;    // FP8 verifier cache: [n_pages][Hkv] fp32 scale of each page's K (V) bytes, else null
  const float* v_scale;
  int max_pages;
  int splits;
  float scale_log2e;
  int wait_limit;          // polls after which a bounded wait gives up: read by the developer build only (MASW_WAIT_LIMIT)
  int early;               // draft (attend_draft_kernel): the counters, slot_pos and this layer's K/V are not written by
                           // the launch's immediate predecessor in the stream, so they may be read before the wait
  int deterministic;       // verify (tcgen05 kernel): every tile assigned statically, results repeat bit for bit
  int next_hint;           // verify (tcgen05 kernel): the second pair of tensor maps names the next call's cache (L2 hint)
  int dt, dm;              // draft: a counter update that was only noted on the host (mem_advance_deferred): the counters in
                           // force are t[b] + dt and min(n_slots[b] + dm, max_slots)
  int guess_hint;          // draft (attend_draft_kernel), launch that may not run ahead: ask the tiles into L2 ahead of the
                           // wait from the counters as they stand (set when the launch's KV is small beside L2)
#ifdef MASW_TRACE
  long long* trace;        // developer build: per-CTA phase timestamps (null = off)
  int drop_tile;           // developer build: the copy of this CTA-local tile is armed but never issued (-1 = off),
                           // which makes a bounded wait run out without any fault
  int debug_flags;         // developer build, draft kernel: 1 = no cross-split reduction, 2 = no tile arithmetic,
                           // 4 = never ahead of the predecessor (timing experiments; results are then meaningless)
#endif
};

struct Segment {
  int phys;   // first entry coordinate inside the (sequence, head) row range
  int len;    // entries
  int xbase;  // index (token position or slot number) of the first entry
  int kind;   // 0 sink, 1 slot, 2 ring / verify cache
};

// Enumerates the contiguous runs of physical entries that some row of this sequence may read.
// Draft (Eq. 3): sink [0,S) | committed (+ pending) slots | the ring pieces holding the union of the
// rows' local windows.  Verify: the cache prefix [0, kv_len).
// HINT: the counters are read with relaxed gpu-scope loads, which leave no line in the SM's own cache: the
// caller runs ahead of a launch that may still be writing them and wants only a guess (for L2 prefetches); it
// reads them again, the ordinary way, once its predecessor has completed.
__device__ __forceinline__ int ld_counter(const int* ptr, bool hint) {
  if (!hint) return *ptr;
  int v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(ptr) : "memory");
  return v;
}
template <bool HINT = false>
__device__ __forceinline__ int build_segments(const AttendParams& p, int b, Segment (&seg)[kMaxSeg], int& t_out,
                                              int& m_out) {
  int n = 0;
  if (p.kv_len != nullptr) {
    int len = min(max(ld_counter(p.kv_len + b, HINT), 0), p.capacity);
    t_out = len;
    m_out = 0;
    if (len > 0) seg[n++] = Segment{0, len, 0, 2};
    return n;
  }
  const int t = max(ld_counter(p.t + b, HINT), 0) + p.dt;
  const int M = min(max(ld_counter(p.n_slots + b, HINT), 0) + p.dm, p.max_slots);
  t_out = t;
  m_out = M;
  const int n_raw = p.n_q - p.last_row_is_slot;
  const int n_tok = t + n_raw;  // raw tokens written so far, pending ones included
  const int ns = min(p.S, n_tok);
  if (ns > 0) seg[n++] = Segment{0, ns, 0, 0};
  const int nsl = min(M + (p.h_g != nullptr ? 0 : p.last_row_is_slot), p.max_slots);   // fused: the pending slot joins in the merge
  if (nsl > 0) seg[n++] = Segment{p.S, nsl, 0, 1};
  const int last0 = t + (n_raw > 0 ? 0 : -1);  // token the first row rides on
  const int a_lo = max(p.S, last0 + 1 - p.W);
  const int a_hi = n_tok - 1;
  if (a_hi >= a_lo) {
    int count = min(a_hi - a_lo + 1, p.ring_cap);
    const int p0 = (a_lo - p.S) % p.ring_cap;
    const int len1 = min(count, p.ring_cap - p0);
    seg[n++] = Segment{p.S + p.max_slots + p0, len1, a_lo, 2};
    if (count > len1) seg[n++] = Segment{p.S + p.max_slots, count - len1, a_lo + len1, 2};
  }
  return n;
}

// ---- tagged partial-result records -----------------------------------------------------------------
// Every value a CTA publishes for the other splits travels as a 64-bit record: the 32-bit payload and the
// 32-bit epoch tag of the launch that wrote it.  A 64-bit access is single-copy atomic, so a reader that
// sees this launch's tag also sees the payload: no fence, flag or atomic is needed between writer and
// reader, and a reader simply reloads a record until its tag is the expected one (bounded).  Both sides use
// relaxed operations at gpu scope: a cache operator (.cg) is only a hint, and a weak load repeated in a tight
// loop may be answered by the SM's own cache for as long as the loop runs.
__device__ __forceinline__ unsigned long long rec_make(float v, int tag) {
  return static_cast<unsigned long long>(__float_as_uint(v)) | (static_cast<unsigned long long>(static_cast<unsigned>(tag)) << 32);
}
__device__ __forceinline__ void rec_store1(unsigned long long* dst, float a, int tag) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(dst), "l"(rec_make(a, tag)) : "memory");
}
__device__ __forceinline__ void rec_store2(unsigned long long* dst, float a, float b, int tag) {   // 16-byte aligned
  asm volatile("st.relaxed.gpu.global.v2.u64 [%0], {%1, %2};" ::"l"(dst), "l"(rec_make(a, tag)), "l"(rec_make(b, tag)) : "memory");
}
struct Rec1 { float a; bool ok; };
struct Rec2 { float a, b; bool ok; };
__device__ __forceinline__ Rec1 rec_load1(const unsigned long long* src, int tag) {
  unsigned long long r;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(r) : "l"(src) : "memory");
  return Rec1{__uint_as_float(static_cast<unsigned>(r)), static_cast<int>(r >> 32) == tag};
}
__device__ __forceinline__ Rec2 rec_load2(const unsigned long long* src, int tag) {   // 16-byte aligned
  unsigned long long r0, r1;
  asm volatile("ld.relaxed.gpu.global.v2.u64 {%0, %1}, [%2];" : "=l"(r0), "=l"(r1) : "l"(src) : "memory");
  return Rec2{__uint_as_float(static_cast<unsigned>(r0)), __uint_as_float(static_cast<unsigned>(r1)),
              static_cast<int>(r0 >> 32) == tag && static_cast<int>(r1 >> 32) == tag};
}

// (m, l) and four o columns of one row of one split
__device__ __forceinline__ void rec_fetch_item(const unsigned long long* ml_rec, const unsigned long long* o_rec, int tag,
                                               float2& ml, float4& v, bool& ok) {
  const Rec2 a = rec_load2(ml_rec, tag);
  const Rec2 b2 = rec_load2(o_rec, tag);
  const Rec2 c2 = rec_load2(o_rec + 2, tag);
  ml = make_float2(a.a, a.b);
  v = make_float4(b2.a, b2.b, c2.a, c2.b);
  ok = a.ok && b2.ok && c2.ok;
}

// Cross-split reduction shared by the attention kernels.  The kernel is launched cooperatively (all CTAs
// co-resident), so the splits of a (sequence, KV head) can consume each other's partials.  Every CTA read
// this head's epoch word in its prologue and published its partial as records tagged epoch + 1.  Here each
// CTA merges its own slice of the (row, 4-column) items out of all splits' records: the items are spread
// over kGroups thread groups, group g taking splits g, g + kGroups, ...; a record whose tag is not yet
// epoch + 1 is reloaded (bounded); the group partials are combined in group order through shared memory, so
// the summation order is fixed and the result is run-to-run identical.  Split 0 advances the epoch word
// when it is done: by then every split has published something, hence has read the old epoch; the word
// lives on the device, so replaying the launch from a CUDA graph works.
// Must be called by all NTHREADS threads of the CTA; `scratch` is shared memory of at least
// NTHREADS * 24 + 8 * D + 64 bytes.
template <int D, int KROWS, int NTHREADS, int kGroups = 4, int kFetch = 6>
__device__ __forceinline__ void split_reduce_and_store(const AttendParams& p, int b, int kvh, int split, int n_rows,
                                                       int epoch, float* scratch, int tid,
                                                       const double* rope_cs = nullptr, long long* tr = nullptr) {
  constexpr float kNegInf = -INFINITY;
  const int bh = b * p.Hkv + kvh;
  __syncthreads();
  const int tag = epoch + 1;
  const unsigned long long* all_o = p.part_o + static_cast<size_t>(bh) * p.splits * KROWS * D;
  const unsigned long long* all_ml = p.part_ml + static_cast<size_t>(bh) * p.splits * KROWS * 2;
  const int splits = p.splits;
  const int n_items = n_rows * (D / 4);
  const int per = (n_items + splits - 1) / splits;
  const int i_begin = split * per;
  const int my_items = max(0, min(n_items, i_begin + per) - i_begin);
  constexpr int kSlots = NTHREADS / kGroups;   // kGroups thread groups per item, each with kFetch splits' records in flight
  float* gsm = scratch;   // [kGroups][kSlots][6]: m, l, o4
  bool timed_out = false;

  // ---- fused slot materialisation, part 2.  The slot rows (the last G query rows) also attend to the slot
  // being created, which is in nobody's tile: its key and value are formed here from the splits' partial
  // sums (in split order), the key is rotated (angles in double), both are rounded to bf16 exactly as they
  // are stored, and the entry joins the slot rows as one more online-softmax term.  Split 0 stores the new
  // entry at slot index n_slots[b].
  const int first_slot_item = (n_rows - p.G) * (D / 4);
  bool slot_term = false;
  float* kg = gsm + kGroups * kSlots * 6;   // [D] key of the new slot (bf16 values)
  float* vg = kg + D;                       // [D]
  float* sg = vg + D;                       // [G] scaled scores of the slot rows against it (log2 domain)
  if (p.h_g != nullptr && (p.active == nullptr || p.active[b] != 0)) {
    const bool need = (split == 0) || (i_begin + my_items > first_slot_item);
    if (need) {
      slot_term = true;
      const unsigned long long* ps = p.part_slot + static_cast<size_t>(bh) * splits * 2 * D;
      const int warp = tid >> 5, lane = tid & 31;
      // the query values of the slot rows (one warp per row) are fetched before the records are awaited
      constexpr int kQPerLane = D / 32;
      constexpr int kRowsPerWarp = 2;
      float qreg[kRowsPerWarp][kQPerLane];
#pragma unroll
      for (int w = 0; w < kRowsPerWarp; ++w) {
        const int g = warp + w * (NTHREADS / 32);
#pragma unroll
        for (int e = 0; e < kQPerLane; ++e) {
          qreg[w][e] = 0.f;
          if (g < p.G) {
            const __nv_bfloat16* qrow = p.q + ((static_cast<size_t>(b) * p.n_q + (p.n_q - 1)) * p.Hq + kvh * p.G + g) * D;
            qreg[w][e] = __bfloat162float(qrow[lane + 32 * e]);
          }
        }
      }
      // unit u < D/2: key columns (u, u + D/2), rotated together; unit D/2 + j: value columns (2j, 2j + 1).
      // Eight splits of both columns are in flight at a time; the sums run in split order.
      for (int u = tid; u < D; u += NTHREADS) {
        const bool is_k = u < D / 2;
        const int c0 = is_k ? u : D + 2 * (u - D / 2);
        const int c1 = is_k ? u + D / 2 : c0 + 1;
        float sum0 = 0.f, sum1 = 0.f;
        for (int sp0 = 0; sp0 < splits; sp0 += 8) {
          float v0[8], v1[8];
          bool ok0[8], ok1[8];
          bool all_ok = true;
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            v0[e] = 0.f; v1[e] = 0.f; ok0[e] = true; ok1[e] = true;
            if (sp0 + e < splits) {
              const unsigned long long* rec = ps + static_cast<size_t>(sp0 + e) * 2 * D;
              const Rec1 r0 = rec_load1(rec + c0, tag), r1 = rec_load1(rec + c1, tag);
              v0[e] = r0.a; ok0[e] = r0.ok; v1[e] = r1.a; ok1[e] = r1.ok;
              all_ok &= r0.ok && r1.ok;
            }
          }
          for (int it = 0; !all_ok && it < MASW_WAIT_LIMIT(p); ++it) {   // a split that has not published yet
            __nanosleep(20);
            all_ok = true;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
              const unsigned long long* rec = ps + static_cast<size_t>(sp0 + e) * 2 * D;
              if (!ok0[e]) { const Rec1 r0 = rec_load1(rec + c0, tag); v0[e] = r0.a; ok0[e] = r0.ok; all_ok &= r0.ok; }
              if (!ok1[e]) { const Rec1 r1 = rec_load1(rec + c1, tag); v1[e] = r1.a; ok1[e] = r1.ok; all_ok &= r1.ok; }
            }
          }
          timed_out |= !all_ok;
#pragma unroll
          for (int e = 0; e < 8; ++e) { sum0 += v0[e]; sum1 += v1[e]; }
        }
        if (is_k) {
          double cs, sn;
          if (rope_cs != nullptr) {
            cs = rope_cs[2 * u];
            sn = rope_cs[2 * u + 1];
          } else {
            const double theta = static_cast<double>(p.slot_pos[b]) * pow(p.rope_base, -2.0 * u / D);
            sincos(theta, &sn, &cs);
          }
          const double x1 = sum0, x2 = sum1;
          sum0 = static_cast<float>(x1 * cs - x2 * sn);
          sum1 = static_cast<float>(x2 * cs + x1 * sn);
        }
        kg[c0] = __bfloat162float(__float2bfloat16_rn(sum0));   // kg | vg are contiguous; values as stored
        kg[c1] = __bfloat162float(__float2bfloat16_rn(sum1));
      }
      __syncthreads();
      // scores of the G slot rows: one warp per row
#pragma unroll
      for (int w = 0; w < kRowsPerWarp; ++w) {
        const int g = warp + w * (NTHREADS / 32);
        if (g < p.G) {
          float dot = 0.f;
#pragma unroll
          for (int e = 0; e < kQPerLane; ++e) dot = fmaf(qreg[w][e], kg[lane + 32 * e], dot);
          for (int o2 = 16; o2 > 0; o2 >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o2);
          if (lane == 0) sg[g] = dot * p.scale_log2e;
        }
      }
      for (int g = warp + kRowsPerWarp * (NTHREADS / 32); g < p.G; g += NTHREADS / 32) {   // very wide groups
        const __nv_bfloat16* qrow = p.q + ((static_cast<size_t>(b) * p.n_q + (p.n_q - 1)) * p.Hq + kvh * p.G + g) * D;
        float dot = 0.f;
        for (int d = lane; d < D; d += 32) dot = fmaf(__bfloat162float(qrow[d]), kg[d], dot);
        for (int o2 = 16; o2 > 0; o2 >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o2);
        if (lane == 0) sg[g] = dot * p.scale_log2e;
      }
      if (split == 0) {
        const int m_slot = p.n_slots[b] + p.dm;
        if (m_slot < p.max_slots) {
          for (int c = tid; c < 2 * D; c += NTHREADS) {
            __nv_bfloat16* dst = (c < D ? p.k_base : p.v_base) + b * p.stride_b + kvh * p.stride_h +
                                 static_cast<long long>(p.S + m_slot) * D + (c % D);
            *dst = __float2bfloat16_rn(kg[c]);
          }
        } else if (tid == 0 && p.status) {
          atomicOr(p.status, MASW_STATUS_SLOT_OVERFLOW);
        }
      }
      __syncthreads();
    }
  }

  for (int base = 0; base < my_items; base += kSlots) {
    const int li = base + tid / kGroups;      // local item
    const int grp = tid % kGroups;
    const bool live = li < my_items;
    const int idx = i_begin + (live ? li : 0);
    const int r = idx / (D / 4);
    const int d4 = (idx % (D / 4)) * 4;
    float m_run2 = kNegInf, l_run2 = 0.f;
    float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
    // everything the final combine needs besides the partials is worked out before the records are awaited,
    // so that little serial work is left once the last split has published
    const int j = r / p.G, g = r % p.G;
    const size_t row_off = (static_cast<size_t>(b) * p.n_q + j) * p.Hq + kvh * p.G + g;
    float* const out_o = p.o + row_off * D + d4;
    __nv_bfloat16* const out_bf16 = p.o_bf16 ? p.o_bf16 + row_off * D + d4 : nullptr;
    float* const out_lse = (d4 == 0 && p.lse) ? p.lse + row_off : nullptr;
    const bool with_slot = slot_term && idx >= first_slot_item;
    const float s_new = with_slot ? sg[g] : 0.f;
    const float4 v_new = with_slot ? make_float4(vg[d4], vg[d4 + 1], vg[d4 + 2], vg[d4 + 3]) : make_float4(0.f, 0.f, 0.f, 0.f);
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
    __syncthreads();
  }
  if (timed_out && p.status) atomicOr(p.status, MASW_STATUS_WAIT_TIMEOUT);
  // every split has published records tagged with this launch's epoch, so all of them have read the old one
  if (split == 0 && tid == 0) p.tickets[bh * (kMaxSplitsDev + 1)] = tag;
}

template <int D, int MT, int EW, int TE, int NSTAGE>
struct AttendCfg {
  static constexpr int kRows = MT * 16;
  static constexpr int kConsumerWarps = MT * EW;
  static constexpr int kThreads = (kConsumerWarps + 1) * 32;
  static constexpr int kSub = D / 64;                 // 128-byte column groups
  static constexpr int kSubBytes = TE * 128;          // one [TE x 64] bf16 box
  static constexpr int kTileBytes = kSub * kSubBytes; // K or V tile
  static constexpr int kStageBytes = 2 * kTileBytes;
  static constexpr int kQSubBytes = kRows * 128;
  static constexpr int kQBytes = kSub * kQSubBytes;
  static constexpr int kPipeBytes = NSTAGE * kStageBytes;
  static constexpr int kMergeStride = D + 8;   // floats per partial row in shared memory (+8: the quad rows land in different banks)
  static constexpr int kMergeBytes = EW * kRows * (kMergeStride + 2) * 4;
  static constexpr int kRopeOff = 2 * NSTAGE * 8 + 64 * 4 + 2 * kMaxSeg * kRows * 4;   // (cos, sin) of the new slot's angles
  static constexpr int kCtrlBytes = kRopeOff + (D / 2) * 16 + 64;
  static constexpr int kSmemBytes = 1024 + kPipeBytes + kQBytes + kCtrlBytes;
  static_assert(kMergeBytes <= kPipeBytes, "merge scratch must fit in the pipeline stages");
  static_assert(D == 64 || D == 128, "head_dim");
  static_assert(TE % 16 == 0 && TE >= 16, "tile entries");
  // Tile i lives in stage i % NSTAGE and is consumed by the warps with ew == i % EW.  With NSTAGE a
  // multiple of EW a stage is always consumed by the same warps, so each warp meets the phases of a
  // stage's barrier strictly in order; otherwise a warp could test a parity two phases ahead of the
  // barrier and read a tile that has not landed.
  static_assert(NSTAGE % EW == 0, "NSTAGE must be a multiple of EW");
};

template <int D, int MT, int EW, int TE, int NSTAGE, int CT>
__global__ void __launch_bounds__((MT * EW + 1) * 32, CT)
attend_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const AttendParams p) {
  using C = AttendCfg<D, MT, EW, TE, NSTAGE>;
  constexpr int kRows = C::kRows;
  constexpr float kNegInf = -INFINITY;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* pipe = smem;
  uint8_t* q_smem = smem + C::kPipeBytes;
  uint8_t* ctrl = q_smem + C::kQBytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(ctrl);
  uint64_t* empty_bar = full_bar + NSTAGE;
  int* plan = reinterpret_cast<int*>(empty_bar + NSTAGE);  // 64 ints
  int* row_lo = plan + 64;                                  // [kMaxSeg][kRows]
  int* row_hi = row_lo + kMaxSeg * kRows;
  double* rope_cs = reinterpret_cast<double*>(ctrl + C::kRopeOff);   // [D/2][2]
  // plan layout: [0] nseg, [1] tile_begin, [2] tile_end, [3] error flag, [4] last-CTA flag
  //              [5] tiles issued by the producer; [6] reduction epoch; [7] committed tokens t; [8+4s..] phys,len,xbase,kind ;
  //              [32+s] first tile of segment s (s = 0..nseg)

  const int tid = threadIdx.x;
  const int warp = tid >> 5;
  const int lane = tid & 31;
  const int split = blockIdx.x;
  const int kvh = blockIdx.y;
  const int b = blockIdx.z;
  const int n_rows = p.n_q * p.G;  // real query rows of this KV head

#ifdef MASW_TRACE
  long long* tr = p.trace ? p.trace + (static_cast<size_t>((blockIdx.z * gridDim.y + blockIdx.y) * gridDim.x + blockIdx.x)) * kTraceWords : nullptr;
#endif
  MASW_STAMP(tr, 0);
  const bool is_producer = (tid == C::kConsumerWarps * 32);   // lane 0 of the producer warp
  if (is_producer) {
    prefetch_tensormap(&tmK);   // the descriptor fetches overlap the barrier setup and the counter loads
    prefetch_tensormap(&tmV);
    for (int s = 0; s < NSTAGE; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], MT);
    }
    fence_mbar_init();
  }

  // everything above touched no global memory: a launch that was allowed to start early waits here for its
  // predecessor, and lets its own successor start
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  // ---- issue the Q loads first so that their latency overlaps the counter loads of the plan
  constexpr int kChunksPerRow = D / 8;  // 16-byte chunks
  constexpr int kQPerThread = (kRows * kChunksPerRow + C::kThreads - 1) / C::kThreads;
  uint4 qv[kQPerThread];
#pragma unroll
  for (int k = 0; k < kQPerThread; ++k) {
    const int idx = tid + k * C::kThreads;
    const int r = idx / kChunksPerRow, cg = idx % kChunksPerRow;
    qv[k] = make_uint4(0, 0, 0, 0);
    if (idx < kRows * kChunksPerRow && r < n_rows) {
      const int j = r / p.G, g = r % p.G;
      const size_t off = ((static_cast<size_t>(b) * p.n_q + j) * p.Hq + kvh * p.G + g) * D + cg * 8;
      qv[k] = __ldg(reinterpret_cast<const uint4*>(p.q + off));
    }
  }

  // ---- plan: segments, this CTA's tile range, per-row visibility bounds
  {
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
      plan[4] = 0;
      plan[7] = t_b;
      plan[6] = __ldcg(p.tickets + (b * p.Hkv + kvh) * (kMaxSplitsDev + 1));   // this head's reduction epoch
    }
    if (is_producer) {
      // the producer plans its own tile range from the same segments and puts the first ring of tiles in
      // flight before the CTA-wide barrier: the first HBM round trip overlaps the rest of the prologue
      int first[kMaxSeg + 1];
      int acc = 0;
      for (int s = 0; s < nseg; ++s) { first[s] = acc; acc += (seg[s].len + TE - 1) / TE; }
      first[nseg] = acc;
      const int tb = static_cast<int>((static_cast<long long>(acc) * split) / p.splits);
      const int te = static_cast<int>((static_cast<long long>(acc) * (split + 1)) / p.splits);
      const uint64_t policy = l2_policy_evict_first();
      int sg = 0;
      for (int i = 0; i < min(te - tb, NSTAGE); ++i) {
        const int it = tb + i;
        while (sg + 1 < nseg && it >= first[sg + 1]) ++sg;
        const int row0 = seg[sg].phys + (it - first[sg]) * TE;
        uint8_t* kdst = pipe + i * C::kStageBytes;
        uint8_t* vdst = kdst + C::kTileBytes;
        mbar_arrive_expect_tx(&full_bar[i], C::kStageBytes);
#ifdef MASW_TRACE
        if (i == p.drop_tile) continue;
#endif
#pragma unroll
        for (int sub = 0; sub < C::kSub; ++sub)
          tma_load_4d(kdst + sub * C::kSubBytes, &tmK, &full_bar[i], sub * 64, row0, kvh, b, policy);
#pragma unroll
        for (int sub = 0; sub < C::kSub; ++sub)
          tma_load_4d(vdst + sub * C::kSubBytes, &tmV, &full_bar[i], sub * 64, row0, kvh, b, policy);
      }
    }
    if (tid < kRows) {
      const int r = min(tid, n_rows - 1);
      const int j = r / p.G;
      int lo_raw, hi_raw, hi_slot;
      if (p.kv_len != nullptr) {
        lo_raw = 0;
        hi_raw = t_b - p.n_q + j;
        hi_slot = -1;
      } else {
        const int n_raw = p.n_q - p.last_row_is_slot;
        const bool is_slot = p.last_row_is_slot && (j == p.n_q - 1);
        const int last = t_b + (is_slot ? n_raw - 1 : j);
        lo_raw = max(p.S, last + 1 - p.W);
        hi_raw = last;
        hi_slot = m_b - 1 + ((is_slot && p.h_g == nullptr) ? 1 : 0);
      }
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
        row_lo[s * kRows + tid] = lo;
        row_hi[s * kRows + tid] = hi;
      }
    }
  }

  // ---- Q tile -> shared memory (rows beyond the real ones are zero), same 128B swizzle as the KV tiles
#pragma unroll
  for (int k = 0; k < kQPerThread; ++k) {
    const int idx = tid + k * C::kThreads;
    if (idx < kRows * kChunksPerRow) {
      const int r = idx / kChunksPerRow, cg = idx % kChunksPerRow;
      const int sub = cg >> 3, c = cg & 7;
      *reinterpret_cast<uint4*>(q_smem + sub * C::kQSubBytes + r * 128 + ((c ^ (r & 7)) << 4)) = qv[k];
    }
  }
  __syncthreads();
  MASW_STAMP(tr, 1);

  const int nseg = plan[0];
  const int tile_begin = plan[1];
  const int tile_end = plan[2];
  const int n_tiles = tile_end - tile_begin;

  // per-thread running state of the consumer warps
  float acc[D / 8][4];
  float m_run[2] = {kNegInf, kNegInf};
  float l_run[2] = {0.f, 0.f};
#pragma unroll
  for (int i = 0; i < D / 8; ++i) { acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f; }

  if (warp == C::kConsumerWarps) {
    // ================= producer warp: one lane issues the bulk copies =================
    if (lane == 0) {
      const uint64_t policy = l2_policy_evict_first();
      int seg = 0;
      bool ok = true;
      plan[5] = min(n_tiles, NSTAGE);
      for (int i = NSTAGE; i < n_tiles && ok; ++i) {   // the first NSTAGE tiles were issued in the prologue
        const int it = tile_begin + i;
        while (seg + 1 < nseg && it >= plan[32 + seg + 1]) ++seg;
        const int i0 = (it - plan[32 + seg]) * TE;
        const int row0 = plan[8 + 4 * seg] + i0;
        const int stage = i % NSTAGE;
        const int round = i / NSTAGE;
        ok = mbar_wait_bounded(&empty_bar[stage], (round - 1) & 1, MASW_WAIT_LIMIT(p));
        if (!ok) break;
        uint8_t* kdst = pipe + stage * C::kStageBytes;
        uint8_t* vdst = kdst + C::kTileBytes;
        mbar_arrive_expect_tx(&full_bar[stage], C::kStageBytes);
        plan[5] = i + 1;  // tiles issued so far (read only on the give-up path)
#ifdef MASW_TRACE
        if (i == p.drop_tile) continue;
#endif
#pragma unroll
        for (int sub = 0; sub < C::kSub; ++sub) {
          tma_load_4d(kdst + sub * C::kSubBytes, &tmK, &full_bar[stage], sub * 64, row0, kvh, b, policy);
        }
#pragma unroll
        for (int sub = 0; sub < C::kSub; ++sub) {
          tma_load_4d(vdst + sub * C::kSubBytes, &tmV, &full_bar[stage], sub * 64, row0, kvh, b, policy);
        }
      }
      if (!ok) {
        plan[3] = 1;
        if (p.status) atomicOr(p.status, MASW_STATUS_WAIT_TIMEOUT);
      }
    } else if (p.h_g != nullptr) {
      // the idle lanes prepare the rotation of the slot this launch creates (angles in double)
      for (int i = lane - 1; i < D / 2; i += 31) {
        const double theta = static_cast<double>(p.slot_pos[b]) * pow(p.rope_base, -2.0 * i / D);
        double sn, cs;
        sincos(theta, &sn, &cs);
        rope_cs[2 * i] = cs;
        rope_cs[2 * i + 1] = sn;
      }
    }
  } else {
    // ================= consumer warps =================
    const int mt = warp % MT;
    const int ew = warp / MT;
    const int qr = lane >> 2;  // row inside the 16-row block (and +8)
    const int qc = lane & 3;

    // Q fragments for this row block, kept in registers for the whole kernel
    uint32_t qf[D / 16][4];
    {
      const int r = mt * 16 + (lane & 15);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const int cg = ks * 2 + (lane >> 4);
        const int sub = cg >> 3, c = cg & 7;
        ldmatrix_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3],
                    smem_u32(q_smem + sub * C::kQSubBytes + r * 128 + ((c ^ (r & 7)) << 4)));
      }
    }

    const int row_a = mt * 16 + qr, row_b = row_a + 8;
    int seg = -1;
    int cur_seg = 0;
    int lo_a = 1, hi_a = 0, lo_b = 1, hi_b = 0;
    bool ok = true;

    for (int i = ew; i < n_tiles; i += EW) {
      const int it = tile_begin + i;
      while (cur_seg + 1 < nseg && it >= plan[32 + cur_seg + 1]) ++cur_seg;
      if (cur_seg != seg) {
        seg = cur_seg;
        lo_a = row_lo[seg * kRows + row_a]; hi_a = row_hi[seg * kRows + row_a];
        lo_b = row_lo[seg * kRows + row_b]; hi_b = row_hi[seg * kRows + row_b];
      }
      const int i0 = (it - plan[32 + seg]) * TE;
      const int seg_len = plan[8 + 4 * seg + 1];
      const int x0 = plan[8 + 4 * seg + 2] + i0;
      const int stage = i % NSTAGE;
      const uint32_t parity = (i / NSTAGE) & 1;
      // Fused append: the pending raw tokens (positions t .. t + n_raw - 1) are not in memory yet.
      // The warp overwrites their rows of the landed tile in shared memory with the caller's K/V, and
      // the first row block's warp also stores them to the arena for later steps.  Nothing orders that
      // store against this launch's bulk copies, and nothing has to: the rows are replaced here.
      // The caller's rows are requested before the tile is awaited (the first kPre 16-byte chunks per
      // lane, which covers two tokens), so their latency is not added to the tile's.
      constexpr int kPre = 2;
      int pat_lo = 0, pat_per = 0;
      uint4 pre[kPre];
      const int t_b = plan[7];
      const int n_raw = p.n_q - p.last_row_is_slot;
      auto raw_src = [&](int idx, int& which, int& r, int& cg) {
        which = idx / pat_per;
        const int rem = idx % pat_per;
        const int tok = pat_lo + rem / (D / 8);
        cg = rem % (D / 8);
        r = tok - x0;
        return reinterpret_cast<const uint4*>((which ? p.v_raw : p.k_raw) +
                                              ((static_cast<size_t>(b) * n_raw + (tok - t_b)) * p.Hkv + kvh) * D + cg * 8);
      };
      if (p.k_raw != nullptr && plan[8 + 4 * seg + 3] != 1) {
        const int lo = max(x0, t_b), hi = min(x0 + min(TE, seg_len - i0), t_b + n_raw);   // inside this segment only
        if (lo < hi) {
          pat_lo = lo;
          pat_per = (hi - lo) * (D / 8);
#pragma unroll
          for (int u = 0; u < kPre; ++u) {
            const int idx = lane + 32 * u;
            if (idx < 2 * pat_per) {
              int which, r, cg;
              pre[u] = __ldg(raw_src(idx, which, r, cg));
            }
          }
        }
      }

      ok = mbar_wait_bounded(&full_bar[stage], parity, MASW_WAIT_LIMIT(p));
      if (!ok) break;

      uint8_t* ksm = pipe + stage * C::kStageBytes;
      uint8_t* vsm = ksm + C::kTileBytes;
      const uint32_t ks_base = smem_u32(ksm);
      const uint32_t vs_base = smem_u32(vsm);

      const bool patched = pat_per > 0;
      if (patched) {
        const int phys0 = plan[8 + 4 * seg] + i0;
        auto put = [&](int idx, uint4 val) {
          int which, r, cg;
          raw_src(idx, which, r, cg);
          uint8_t* tile = which ? vsm : ksm;
          *reinterpret_cast<uint4*>(tile + (cg >> 3) * C::kSubBytes + r * 128 + (((cg & 7) ^ (r & 7)) << 4)) = val;
          if (mt == 0) {
            __nv_bfloat16* dst = (which ? p.v_base : p.k_base) + b * p.stride_b + kvh * p.stride_h +
                                 static_cast<long long>(phys0 + r) * D + cg * 8;
            *reinterpret_cast<uint4*>(dst) = val;
          }
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

      // entries of the tile beyond the segment hold foreign bytes: zero their V rows so that a
      // zero probability times a non-finite value cannot poison the accumulators
      const int valid = min(TE, seg_len - i0);
      if (valid < TE) {
        for (int idx = lane; idx < (TE - valid) * (D / 8); idx += 32) {
          const int r = valid + idx / (D / 8);
          const int cg = idx % (D / 8);
          *reinterpret_cast<uint4*>(vsm + (cg >> 3) * C::kSubBytes + r * 128 + ((cg & 7) << 4)) = make_uint4(0, 0, 0, 0);
        }
        fence_proxy_async();   // every lane orders its own stores ahead of the next bulk copy into this stage
        __syncwarp();
      }

      // ---- S = Q K^T  (16 rows x TE entries).  The K fragments of step ks + 1 are fetched before the
      // MMAs of step ks are issued, and even / odd steps accumulate into separate registers, so neither
      // the shared-memory latency nor the MMA dependency chain is exposed.
      float s[TE / 8][4], s2[TE / 8][4];
#pragma unroll
      for (int nt = 0; nt < TE / 8; ++nt) {
        s[nt][0] = s[nt][1] = s[nt][2] = s[nt][3] = 0.f;
        s2[nt][0] = s2[nt][1] = s2[nt][2] = s2[nt][3] = 0.f;
      }
      {
        const int mat = lane >> 3, r8 = lane & 7;
        uint32_t kb[2][TE / 16][4];
        auto load_k = [&](int ks, uint32_t (&dst)[TE / 16][4]) {
#pragma unroll
          for (int np = 0; np < TE / 16; ++np) {
            const int e = np * 16 + (mat >> 1) * 8 + r8;
            const int cg = ks * 2 + (mat & 1);
            ldmatrix_x4(dst[np][0], dst[np][1], dst[np][2], dst[np][3],
                        ks_base + (cg >> 3) * C::kSubBytes + e * 128 + (((cg & 7) ^ (e & 7)) << 4));
          }
        };
        load_k(0, kb[0]);
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          if (ks + 1 < D / 16) load_k(ks + 1, kb[(ks + 1) & 1]);
#pragma unroll
          for (int np = 0; np < TE / 16; ++np) {
            if (ks & 1) {
              mma_bf16_16816(s2[2 * np], qf[ks], kb[ks & 1][np][0], kb[ks & 1][np][1]);
              mma_bf16_16816(s2[2 * np + 1], qf[ks], kb[ks & 1][np][2], kb[ks & 1][np][3]);
            } else {
              mma_bf16_16816(s[2 * np], qf[ks], kb[ks & 1][np][0], kb[ks & 1][np][1]);
              mma_bf16_16816(s[2 * np + 1], qf[ks], kb[ks & 1][np][2], kb[ks & 1][np][3]);
            }
          }
        }
#pragma unroll
        for (int nt = 0; nt < TE / 8; ++nt) {
          s[nt][0] += s2[nt][0]; s[nt][1] += s2[nt][1]; s[nt][2] += s2[nt][2]; s[nt][3] += s2[nt][3];
        }
      }

      // ---- scale, mask, online softmax (exp2 domain)
      const int x_last = x0 + TE - 1;
      const bool need_mask = (x0 < max(lo_a, lo_b)) || (x_last > min(hi_a, hi_b));
      float mx_a = kNegInf, mx_b = kNegInf;
#pragma unroll
      for (int nt = 0; nt < TE / 8; ++nt) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float v = s[nt][c] * p.scale_log2e;
          if (need_mask) {
            const int x = x0 + nt * 8 + 2 * qc + (c & 1);
            const bool vis = (c < 2) ? (x >= lo_a && x <= hi_a) : (x >= lo_b && x <= hi_b);
            v = vis ? v : kNegInf;
          }
          s[nt][c] = v;
        }
        mx_a = fmaxf(mx_a, fmaxf(s[nt][0], s[nt][1]));
        mx_b = fmaxf(mx_b, fmaxf(s[nt][2], s[nt][3]));
      }
      mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 1));
      mx_a = fmaxf(mx_a, __shfl_xor_sync(0xffffffffu, mx_a, 2));
      mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 1));
      mx_b = fmaxf(mx_b, __shfl_xor_sync(0xffffffffu, mx_b, 2));
      const float mn_a = fmaxf(m_run[0], mx_a), mn_b = fmaxf(m_run[1], mx_b);
      const float mu_a = (mn_a == kNegInf) ? 0.f : mn_a;
      const float mu_b = (mn_b == kNegInf) ? 0.f : mn_b;
      // the accumulators are rescaled only when some row of the warp saw a new maximum (after the first
      // few tiles that is rare); when none did, every correction factor is exactly 1
      if (__any_sync(0xffffffffu, mn_a != m_run[0] || mn_b != m_run[1])) {
        const float corr_a = fast_exp2(m_run[0] - mu_a), corr_b = fast_exp2(m_run[1] - mu_b);
        m_run[0] = mn_a; m_run[1] = mn_b;
        l_run[0] *= corr_a; l_run[1] *= corr_b;
#pragma unroll
        for (int i2 = 0; i2 < D / 8; ++i2) {
          acc[i2][0] *= corr_a; acc[i2][1] *= corr_a;
          acc[i2][2] *= corr_b; acc[i2][3] *= corr_b;
        }
      }
      // Probabilities go to the tensor cores as bf16.  The row sum is taken over the ROUNDED values so
      // that the result stays an exact convex combination.  A single 16-row block (the draft's decode
      // rows) is cheap on the tensor pipe, so there the rounding residual is fed through a second MMA
      // (p = p_hi + p_lo), which removes the bf16 rounding of p from the result.
      constexpr bool kSplitP = (MT == 1);
      uint32_t pf[TE / 16][4];
      uint32_t pl[kSplitP ? TE / 16 : 1][4];
#pragma unroll
      for (int nt = 0; nt < TE / 8; ++nt) {
        const float p0 = fast_exp2(s[nt][0] - mu_a), p1 = fast_exp2(s[nt][1] - mu_a);
        const float p2 = fast_exp2(s[nt][2] - mu_b), p3 = fast_exp2(s[nt][3] - mu_b);
        const uint32_t ha = pack_bf16x2(p0, p1), hb = pack_bf16x2(p2, p3);
        const float r0 = __uint_as_float(ha << 16), r1 = __uint_as_float(ha & 0xffff0000u);
        const float r2 = __uint_as_float(hb << 16), r3 = __uint_as_float(hb & 0xffff0000u);
        pf[nt >> 1][(nt & 1) * 2 + 0] = ha;
        pf[nt >> 1][(nt & 1) * 2 + 1] = hb;
        if constexpr (kSplitP) {
          l_run[0] += p0 + p1;
          l_run[1] += p2 + p3;
          pl[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16x2(p0 - r0, p1 - r1);
          pl[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16x2(p2 - r2, p3 - r3);
        } else {
          l_run[0] += r0 + r1;
          l_run[1] += r2 + r3;
        }
      }

      // ---- O += P V, V fragments fetched one step ahead of the MMAs that use them
      {
        const int mat = lane >> 3, r8 = lane & 7;
        constexpr int kSteps = (TE / 16) * (D / 16);
        uint32_t vb[2][4];
        auto load_v = [&](int step, uint32_t (&dst)[4]) {
          const int kk = step / (D / 16), dp = step % (D / 16);
          const int e = kk * 16 + (mat & 1) * 8 + r8;
          const int cg = dp * 2 + (mat >> 1);
          ldmatrix_x4_trans(dst[0], dst[1], dst[2], dst[3],
                            vs_base + (cg >> 3) * C::kSubBytes + e * 128 + (((cg & 7) ^ (e & 7)) << 4));
        };
        load_v(0, vb[0]);
#pragma unroll
        for (int step = 0; step < kSteps; ++step) {
          if (step + 1 < kSteps) load_v(step + 1, vb[(step + 1) & 1]);
          const int kk = step / (D / 16), dp = step % (D / 16);
          mma_bf16_16816(acc[2 * dp], pf[kk], vb[step & 1][0], vb[step & 1][1]);
          mma_bf16_16816(acc[2 * dp + 1], pf[kk], vb[step & 1][2], vb[step & 1][3]);
          if constexpr (kSplitP) {
            mma_bf16_16816(acc[2 * dp], pl[kk], vb[step & 1][0], vb[step & 1][1]);
            mma_bf16_16816(acc[2 * dp + 1], pl[kk], vb[step & 1][2], vb[step & 1][3]);
          }
        }
      }

      // release the stage to the producer
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[stage]);
    }
    if (!ok && lane == 0) {
      plan[3] = 1;
      if (p.status) atomicOr(p.status, MASW_STATUS_WAIT_TIMEOUT);
    }
    // row sums were kept per thread: finish them across the quad
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 1);
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], 2);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 1);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], 2);
  }

  __syncthreads();  // every tile consumed (or abandoned): the stages can be reused as merge scratch
  MASW_STAMP(tr, 2);
  if (plan[3] != 0) {
    // give-up path: a wait ran out.  Let this CTA's copies that are still in flight land (bounded)
    // before shared memory is reused or released; the outputs of this launch are not meaningful.
    if (tid == 0) {
      const int issued = plan[5];
      for (int i = max(0, issued - NSTAGE); i < issued; ++i) {
        mbar_wait_bounded(&full_bar[i % NSTAGE], (i / NSTAGE) & 1, MASW_WAIT_LIMIT(p));
      }
    }
    __syncthreads();
  }

  // ---- fused slot materialisation, part 1: this CTA's slice of K_g = h_g W_K,g and V_g = h_g W_V,g for its
  //      KV head (rows [k0, k1) of the d_model contraction); the splits' partial sums are combined, rotated
  //      and used after the rendezvous (split_reduce_and_store).  A thread owns eight columns (one 16-byte
  //      load per weight row) of every kRowLanes-th row, so all of its loads are in flight together.
  if (p.h_g != nullptr) {
    constexpr int kColThreads = D / 8;
    constexpr int kRowLanes = C::kThreads / kColThreads;
    constexpr int kChunk = 8;   // weight rows per thread and round trip
    const bool act = (p.active == nullptr) || (p.active[b] != 0);
    const int k0 = static_cast<int>((static_cast<long long>(p.d_model) * split) / p.splits);
    const int k1 = static_cast<int>((static_cast<long long>(p.d_model) * (split + 1)) / p.splits);
    __nv_bfloat16* hs = reinterpret_cast<__nv_bfloat16*>(pipe);                       // [k1 - k0]
    float* red = reinterpret_cast<float*>(pipe + 16384);                              // [kRowLanes][2 * D]
    if (act) {
      for (int k = k0 + tid; k < k1; k += C::kThreads) hs[k - k0] = p.h_g[static_cast<size_t>(b) * p.d_model + k];
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
            const float x = __bfloat162float(hs[k - k0]);
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
    unsigned long long* pslot = p.part_slot + (static_cast<size_t>(b * p.Hkv + kvh) * p.splits + split) * 2 * D;
    for (int c = tid; c < 2 * D; c += C::kThreads) {
      float a = 0.f;
      for (int l2 = 0; l2 < kRowLanes; ++l2) a += red[l2 * 2 * D + c];
      rec_store1(pslot + c, a, plan[6] + 1);
    }
    __syncthreads();   // the staging area is reused below
  }

  // ---- per-warp partials -> shared memory
  constexpr int kMS = C::kMergeStride;
  float* mo = reinterpret_cast<float*>(pipe);              // [EW][kRows][kMS]
  float* mml = mo + EW * kRows * kMS;                      // [EW][kRows][2]
  if (warp < C::kConsumerWarps) {
    const int mt = warp % MT, ew = warp / MT;
    const int qr = lane >> 2, qc = lane & 3;
    const int ra = mt * 16 + qr, rb = ra + 8;
    float* oa = mo + (ew * kRows + ra) * kMS;
    float* ob = mo + (ew * kRows + rb) * kMS;
#pragma unroll
    for (int nt = 0; nt < D / 8; ++nt) {
      *reinterpret_cast<float2*>(oa + nt * 8 + 2 * qc) = make_float2(acc[nt][0], acc[nt][1]);
      *reinterpret_cast<float2*>(ob + nt * 8 + 2 * qc) = make_float2(acc[nt][2], acc[nt][3]);
    }
    if (qc == 0) {
      mml[(ew * kRows + ra) * 2 + 0] = m_run[0]; mml[(ew * kRows + ra) * 2 + 1] = l_run[0];
      mml[(ew * kRows + rb) * 2 + 0] = m_run[1]; mml[(ew * kRows + rb) * 2 + 1] = l_run[1];
    }
  }
  __syncthreads();

  // ---- merge the EW partials of each row into this split's partial
  const int bh = b * p.Hkv + kvh;
  unsigned long long* po = p.part_o + (static_cast<size_t>(bh) * p.splits + split) * kRows * D;
  unsigned long long* pml = p.part_ml + (static_cast<size_t>(bh) * p.splits + split) * kRows * 2;
  const int tag = plan[6] + 1;   // this launch's epoch tag
  for (int idx = tid; idx < n_rows * (D / 4); idx += C::kThreads) {
    const int r = idx / (D / 4);
    const int d4 = (idx % (D / 4)) * 4;
    float m = kNegInf;
#pragma unroll
    for (int e = 0; e < EW; ++e) m = fmaxf(m, mml[(e * kRows + r) * 2]);
    float4 o4 = make_float4(0.f, 0.f, 0.f, 0.f);
    float l = 0.f;
#pragma unroll
    for (int e = 0; e < EW; ++e) {
      const float me = mml[(e * kRows + r) * 2];
      const float w = (me == kNegInf) ? 0.f : fast_exp2(me - m);
      const float4 v = *reinterpret_cast<const float4*>(mo + (e * kRows + r) * kMS + d4);
      o4.x += w * v.x; o4.y += w * v.y; o4.z += w * v.z; o4.w += w * v.w;
      l += w * mml[(e * kRows + r) * 2 + 1];
    }
    rec_store2(po + r * D + d4, o4.x, o4.y, tag);
    rec_store2(po + r * D + d4 + 2, o4.z, o4.w, tag);
    if (d4 == 0) rec_store2(pml + r * 2, m, l, tag);
  }

  // ---- cross-split reduction (see split_reduce_and_store)
  MASW_STAMP(tr, 3);
#ifdef MASW_TRACE
  if (tr && tid == 0) { tr[5] = 1; tr[6] = n_tiles; unsigned sm; asm("mov.u32 %0, %%smid;" : "=r"(sm)); tr[7] = sm; }
#endif
  split_reduce_and_store<D, kRows, C::kThreads>(p, b, kvh, split, n_rows, plan[6], reinterpret_cast<float*>(pipe), tid,
                                                p.h_g != nullptr ? rope_cs : nullptr);
  MASW_STAMP(tr, 4);
}

}  // namespace masw
