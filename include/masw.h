/*
 * masw.h — C ABI of the MASW hot-path library for NVIDIA B200 (sm_100a).
 *
 * The library implements, as hand-written CUDA kernels, the data-parallel hot path of
 * memory-augmented sliding-window (MASW) drafting for long-context speculative decoding
 * (arXiv 2608.30252):
 *
 *   mem_init / mem_load / mem_update / mem_advance / mem_rollback   the draft's three-part KV memory
 *   draft_attend                                                   decode attention over that memory
 *   verify_attend                                                  the verifier's attention over its full cache
 *   accept_reject                                                  the standard accept/reject rule
 *
 * Conventions that hold for every entry point
 *   - Pointers marked [device] are device addresses, [host] are host addresses.  The caller owns every
 *     device buffer (KV arena, caches, q/o, logits, workspaces); the library owns only the small host
 *     handle returned by mem_init.  Device pointers must be 16-byte aligned.
 *   - bf16 tensors are passed as `const void*` / `void*` (16-bit brain-float, little endian).
 *   - Every call is asynchronous on `stream` (a cudaStream_t passed as void*); the library never
 *     synchronises the stream except where a function says it does.  Calls that share a workspace
 *     must be ordered on one stream (or by events); overlapping them on the GPU is a race.
 *   - Arguments are validated on the host before anything is launched.  Return value 0 is success;
 *     negative values are the MASW_E* codes below and masw_last_error() describes the failure.
 *   - Device-side conditions that the host cannot see in advance (a full slot region, a wait on one of
 *     the kernel's own copies that ran out) never trap: the kernel records a bit in a status word,
 *     skips the offending access and returns.  mem_get_state reads the draft memory's word back;
 *     verify_attend and accept_reject take a status pointer of their own.  After MASW_STATUS_WAIT_TIMEOUT
 *     the outputs of that launch are meaningless; the next launch on the same workspace is sound again.
 *   - There is no CPU fallback: without a CUDA device every compute entry point fails with MASW_ECUDA.
 *
 * Positions are 0-based: the paper's token i (1-based) is index i-1.
 */
#ifndef MASW_H_
#define MASW_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  MASW_OK = 0,
  MASW_EINVAL = -1,     /* bad argument (NULL, out of range, unsupported head_dim / group size) */
  MASW_EALIGN = -2,     /* a device pointer or stride is not 16-byte aligned */
  MASW_ECAPACITY = -3,  /* slot region, ring or workspace too small for the request */
  MASW_ESTATE = -4,     /* call order violated (e.g. draft_attend with more pending rows than appended) */
  MASW_ECUDA = -5       /* CUDA runtime / driver error, or no device */
};

/* bits of the device status word */
enum {
  MASW_STATUS_SLOT_OVERFLOW = 1,   /* a slot append was skipped: slot region full */
  MASW_STATUS_WAIT_TIMEOUT = 2,    /* a bounded wait on the kernel's own bulk copies gave up */
  MASW_STATUS_BAD_LOGIT = 4,       /* accept_reject met a NaN or infinite logit (a -inf mask included), or, when sampling,
                                      |logit / temperature| too large */
  MASW_STATUS_BAD_TOKEN = 8        /* accept_reject met a draft token outside [0, V) */
};

/* regions of the draft memory (Eq. 3: M_t = M_sink u M_local,t u M_slot,t) */
enum { MASW_REGION_SINK = 0, MASW_REGION_SLOT = 1, MASW_REGION_LOCAL = 2 };

typedef struct masw_mem masw_mem; /* opaque host handle */

/* Geometry of the draft model's attention and of its working memory (Section 4.1; Section 5.1 gives
 * the paper's constants S = W = 128, rollback 16, r = 4 or 8). */
typedef struct masw_config {
  int32_t n_layers;      /* draft transformer layers; each has its own K/V memory */
  int32_t batch;         /* sequences B */
  int32_t n_q_heads;     /* Hq */
  int32_t n_kv_heads;    /* Hkv; query head h reads KV head h / (Hq / Hkv) */
  int32_t head_dim;      /* D: 64 or 128 */
  int32_t d_model;       /* width of the slot hidden state h_g (rows of W_K,g / W_V,g) */
  int32_t sink;          /* S: first S raw tokens, never evicted */
  int32_t window;        /* W: local-window width (most recent non-sink raw tokens that stay visible) */
  int32_t slot_interval; /* r: one memory slot per r non-sink raw tokens (informative; the caller decides when a boundary fires) */
  int32_t rollback;      /* raw tokens physically retained beyond the window so a rollback can re-expose them */
  int32_t max_slots;     /* capacity of the append-only slot region */
  int32_t gamma_max;     /* largest number of pending (uncommitted) raw tokens per sequence */
  float softmax_scale;   /* 0 selects 1 / sqrt(D) */
  float rope_base;       /* 0 selects 500000; slot keys are rotated with theta_i = pos * base^(-2i/D), pairs (i, i + D/2) */
} masw_config;

/* Description of the verifier's (caller-owned) KV cache: element strides, in bf16 elements, of
 * K and V laid out [batch][kv head][entry][head_dim] with head_dim contiguous. */
typedef struct masw_kv_desc {
  const void* k;             /* [device] bf16 */
  const void* v;             /* [device] bf16 */
  int64_t stride_b;          /* elements between sequences; multiple of 8 */
  int64_t stride_h;          /* elements between KV heads; multiple of 8 */
  int64_t stride_n;          /* elements between cache entries; multiple of 8, >= head_dim */
  int32_t batch, n_q_heads, n_kv_heads, head_dim; /* head_dim 64 or 128 */
  int32_t capacity;          /* entries allocated per (sequence, head) */
  const int32_t* kv_len;     /* [device] [batch] entries in use, INCLUDING the T rows being verified */
  float softmax_scale;       /* 0 selects 1 / sqrt(D) */
  int32_t flags;             /* MASW_KV_* bits, 0 for the defaults */
  int32_t* status;           /* [device] one int32 that receives MASW_STATUS_* bits (OR-ed in), or NULL */
  const void* next_k;        /* [device] optional hint (verify_attend, head_dim 128): K and V of the cache the NEXT call */
  const void* next_v;        /*   will read (the next layer's; same geometry and strides), or NULL.  When its own tiles
                                  are all requested, each CTA asks for the first tile it will stream in that call to be
                                  brought into L2, so the next launch does not start on a cold DRAM round trip.  Only a
                                  hint: nothing is read through these pointers. */
} masw_kv_desc;

/* masw_kv_desc.flags / masw_paged_kv_desc.flags */
enum {
  /* verify_attend, head_dim 128: assign every KV tile to its split statically instead of letting the splits
   * of a head claim tiles from a shared pool.  A repeated call on the same inputs then returns the same
   * bits (the pooled schedule only agrees within the rounding of the bf16 probabilities), a little slower
   * because every split waits for the slowest SM. */
  MASW_KV_DETERMINISTIC = 1,
  /* verify_attend, head_dim 128, contiguous cache: the caller vouches that the kernel which precedes this call
   * in the stream writes nothing of the K and V arrays nor of kv_len (the T new rows were appended and the
   * lengths set by an earlier kernel, as they are for every layer but the first of a verification pass, or the
   * cache is static as in a benchmark).  The launch may then read kv_len and request its first K/V tiles (a
   * whole ring of them) before it waits for that kernel; q and the scratch are still read behind the wait.
   * Without the flag everything is read behind the wait. */
  MASW_KV_STABLE = 2
};

/* ---------------------------------------------------------------------------------------------------
 * Sizing.  Host only, no CUDA call.
 * kv_arena_bytes: bytes of the draft KV arena, laid out [layer][K|V][batch][kv head][entry][D] bf16 with
 *   per-(sequence, head) entries = [0,S) sink | [S, S+max_slots) slots | ring of W + rollback + gamma_max
 *   raw tokens rounded up to 64 (Section 4.1's three parts kept as three contiguous regions; the order
 *   of entries does not matter to softmax attention).
 * workspace_bytes: scratch for per-sequence counters, status word, split-K partials and tickets. */
int masw_sizes(const masw_config* cfg, size_t* kv_arena_bytes, size_t* workspace_bytes);

/* Creates the draft memory (Eq. 3) over caller-owned device buffers; zeroes the arena and the
 * workspace on `stream`.  *out receives the handle.  Needs a CUDA device (builds TMA descriptors). */
int mem_init(const masw_config* cfg, void* kv_arena /*[device]*/, size_t kv_arena_bytes,
             void* workspace /*[device]*/, size_t workspace_bytes, void* stream, masw_mem** out);

/* Frees the host handle only. */
void mem_free(masw_mem* mem);

/* Imports already-computed K/V into one region of one layer (the result of the draft-side prefill of
 * Section 4.3, which is outside this library).  k, v: [device] bf16 with element strides
 * strides[0] (sequence), strides[1] (entry), strides[2] (kv head), head_dim contiguous.
 * `first` is the index of the first imported entry inside the region: a sink position, a slot index,
 * or, for MASW_REGION_LOCAL, a raw-token position (>= S; it lands in the ring at (pos - S) mod ring). */
int mem_load(masw_mem* mem, int layer, int region, const void* k, const void* v, int first, int n,
             const int64_t strides[3], void* stream);

/* Sets / reads the per-sequence counters: t[b] = committed raw tokens, n_slots[b] = committed slots.
 * Host arrays of length batch.  mem_set_state enqueues on `stream`; mem_get_state synchronises
 * `stream` and also returns the status word (any of t, n_slots, status may be NULL).  Status bits
 * accumulate on the device between reads; a read with status != NULL returns them and clears the word. */
int mem_set_state(masw_mem* mem, const int32_t* t /*[host]*/, const int32_t* n_slots /*[host]*/, void* stream);
int mem_get_state(masw_mem* mem, int32_t* t /*[host]*/, int32_t* n_slots /*[host]*/, int32_t* status /*[host]*/, void* stream);

/* One layer's share of the memory update cycle (Section 4.2, "Projection and KV materialization" and
 * "Memory update cycle").  Either part may be absent (NULL pointers):
 *  (i)  k_raw, v_raw [device] bf16 [batch][n_raw][Hkv][D]: K/V of the step's raw tokens (already
 *       position-encoded by the backbone).  Token t[b]+i is written to the sink region while its
 *       position is < S, else to the ring.  The tokens stay pending until mem_advance.
 *  (ii) h_g [device] bf16 [batch][d_model], Wk_g, Wv_g [device] bf16 [d_model][Hkv*D] row-major: the
 *       slot token's hidden state and the layer's mirrored projections.  Computes
 *       K_g = RoPE(h_g Wk_g, slot_pos[b]), V_g = h_g Wv_g (fp32 accumulation, rounded to bf16) and
 *       writes them at slot index n_slots[b] for every sequence with active[b] != 0.
 *       slot_pos [device] int32 [batch]: position id of the raw token that follows the slot (the slot
 *       shares that id).  active [device] uint8 [batch] or NULL (all active): sequences not at a
 *       boundary skip the slot (Section 5.1, heterogeneous batches).  The slot stays pending (visible
 *       only to a slot row of draft_attend) until mem_advance(..., add_slot = 1).
 * Nothing older is edited in place and nothing is copied on eviction: eviction is the window start
 * moving when mem_advance bumps t.  Returns MASW_ECAPACITY if the host-side bound on the slot count
 * says the region is full. */
int mem_update(masw_mem* mem, int layer, const void* k_raw, const void* v_raw, int n_raw,
               const void* h_g, const void* Wk_g, const void* Wv_g, const int32_t* slot_pos,
               const uint8_t* active, void* stream);

/* Once per draft step, after every layer was updated: t[b] += n_tokens and, if add_slot != 0,
 * n_slots[b] += 1 for every sequence with active[b] != 0 (active [device] or NULL = all). */
int mem_advance(masw_mem* mem, int n_tokens, int add_slot, const uint8_t* active, void* stream);

/* The same counter update for all sequences (no `active` mask), noted on the host only: nothing is launched
 * and nothing on the device changes.  The draft attention calls that follow and mem_rollback take the noted
 * amounts as launch parameters (t[b] + pending tokens, min(n_slots[b] + pending slots, max_slots) are the
 * counters in force); every other call that reads or writes the counters (mem_get_state, mem_set_state,
 * mem_update, mem_load, mem_advance, draft_prefill_attend) first applies them with one launch, as mem_flush
 * does.  What it buys (Section 4.3: the draft runs L_draft steps back to back): no counter kernel between
 * draft steps, and the first layer's launch of the next step may run ahead of its predecessor like any other
 * layer's, because no launch in between writes the counters.  Several deferred updates accumulate.
 * CUDA graphs: the amounts are baked into the launches that are recorded after this call, so a graph must
 * contain the whole span from the first deferred update to the call that applies it (mem_rollback,
 * mem_flush, ...), and the handle must have nothing pending when the recording starts.
 * Returns MASW_ECAPACITY if the host-side bound on the slot count says the region is full; a slot count that
 * would exceed max_slots on the device is clamped and reported (MASW_STATUS_SLOT_OVERFLOW) when applied. */
int mem_advance_deferred(masw_mem* mem, int n_tokens, int add_slot);

/* Applies what mem_advance_deferred noted (one small launch on `stream`; nothing when nothing is pending). */
int mem_flush(masw_mem* mem, void* stream);

/* Section 4.3, "Rollback": after a rejection drop the speculative raw tokens and the slots created
 * after the last accepted position.  t_keep, slots_keep [device] int32 [batch]: the new counters
 * (t_keep[b] <= t[b], not more than `rollback` + gamma_max tokens back; slots_keep[b] <= n_slots[b]).
 * slots_keep_max [host value]: an upper bound on slots_keep[] that refreshes the host-side capacity
 * check (pass -1 to leave it unchanged).
 * Raw KV inside the retained rollback window becomes visible again; no data moves. */
int mem_rollback(masw_mem* mem, const int32_t* t_keep, const int32_t* slots_keep, int slots_keep_max, void* stream);

/* Draft decode attention over the compact memory (Section 4.1, Eq. 3 and the definition of
 * M_local,t; Section 4.2 for the slot row).  q [device] bf16 [batch][n_q][Hq][D], already
 * position-encoded.  Rows 0 .. n_raw-1 (n_raw = n_q - last_row_is_slot) are the pending raw tokens
 * t[b] .. t[b]+n_raw-1 appended by mem_update; row j sees the sink entries, the n_slots[b] committed
 * slots and the last W non-sink raw tokens up to and including token t[b]+j.  If last_row_is_slot,
 * the last row is the memory-slot token inserted after the last raw row: it sees what that raw row
 * sees plus its own pending slot entry.  Outputs: o [device] fp32 [batch][n_q][Hq][D];
 * lse [device] fp32 [batch][n_q][Hq] (natural-log sum of exp of the scaled scores) or NULL;
 * o_bf16 [device] bf16 copy of o or NULL.  n_q * (Hq/Hkv) must be <= 64 (and n_q - last_row_is_slot <= gamma_max). */
int draft_attend(masw_mem* mem, int layer, const void* q, int n_q, int last_row_is_slot,
                 float* o, float* lse, void* o_bf16, void* stream);

/* mem_update's raw-token append and draft_attend in one launch (Section 4.2: the raw K/V is appended
 * in the same draft pass that attends over it).  k_raw, v_raw [device] bf16 [batch][n_raw][Hkv][D] with
 * n_raw = n_q - last_row_is_slot >= 1: the K/V of the pending raw tokens t[b] .. t[b]+n_raw-1.  The
 * result equals mem_update(layer, k_raw, v_raw, n_raw, ...) followed by draft_attend(...): the tokens
 * are stored in the memory (sink region or ring) for later steps and take part in this call's
 * attention.  A pending slot, if any, must already have been written by mem_update. */
int draft_append_attend(masw_mem* mem, int layer, const void* k_raw, const void* v_raw, const void* q,
                        int n_q, int last_row_is_slot, float* o, float* lse, void* o_bf16, void* stream);

/* The whole boundary step of one layer in one launch (Section 4.2: the slot token is run through the layer
 * together with the raw token, its K/V is appended in the same pass): raw-token append, slot
 * materialisation K_g = RoPE(h_g Wk_g, slot_pos[b]), V_g = h_g Wv_g (fp32 accumulation, bf16 store at slot
 * index n_slots[b], sequences with active[b] == 0 skipped), and the attention of the n_q - 1 raw rows and
 * of the slot row (the last row of q), which also sees the slot it creates.  Arguments as in mem_update
 * and draft_attend; the result equals mem_update(raw) + mem_update(slot) + draft_attend(last_row_is_slot = 1).
 * Follow it, after all layers, with mem_advance(n_q - 1, add_slot = 1, active). */
int draft_boundary_attend(masw_mem* mem, int layer, const void* k_raw, const void* v_raw, const void* h_g,
                          const void* Wk_g, const void* Wv_g, const int32_t* slot_pos, const uint8_t* active,
                          const void* q, int n_q, float* o, float* lse, void* o_bf16, void* stream);

/* Number of memory slots created while a prefix of P raw tokens is processed: floor((P - S) / r) for
 * P > S, else 0 (Section 4.2, boundary every r non-sink tokens).  Host only; -1 on a bad argument. */
int draft_prefill_slots(const masw_config* cfg, int P);

/* The draft's prefill pass of one layer with the structured memory mask (Section 4.3 "Prefill";
 * Appendix C): one launch gives the attention output of every raw prefix token and of every memory-slot
 * token created inside the prefix, so the initial memory is built without exposing ordinary tokens to the
 * full raw history.  Rows and entries are numbered alike: the P raw tokens in order, followed by the
 * M = draft_prefill_slots(cfg, P) slot tokens (slot m, m = 1..M, at index P + m - 1; it was inserted
 * after raw token S + m r - 1, 0-based).
 *   raw token t attends to: sinks [0, min(S, t + 1)), slots 1..floor((t - S) / r), raw tokens
 *     max(S, t + 1 - W)..t;
 *   slot m attends to: sinks [0, S), slots 1..m (itself included), raw tokens max(S, tau + 1 - W)..tau with
 *     tau = S + m r - 1.
 * kv: K and V [device] bf16 of those P + M entries (keys position-encoded), described by element strides;
 *   batch, heads and head_dim must equal the memory's configuration, capacity >= P + M; kv_len is ignored.
 *   Values must be finite.
 * q [device] bf16 [batch][P + M][Hq][D]; o fp32 and/or o_bf16 [batch][P + M][Hq][D] (either may be NULL, not
 * both), lse fp32 [batch][P + M][Hq] or NULL.  Hq / Hkv must divide 128.
 * import_memory != 0: the launch is followed by copies of the sinks, all M slots and the last
 *   min(P - S, W + rollback) raw tokens into this layer's regions of the arena; after the last layer the
 *   caller sets the counters with mem_set_state(t = P, n_slots = M). */
int draft_prefill_attend(masw_mem* mem, int layer, const masw_kv_desc* kv, const void* q, int P, float* o, float* lse,
                         void* o_bf16, int import_memory, void* stream);

/* Bytes of scratch verify_attend needs for this cache geometry and up to T rows.  Host only.
 * The scratch must be zero-filled once before its first use; every call leaves it reusable. */
size_t verify_workspace_bytes(const masw_kv_desc* kv, int T);

/* The verifier's attention over its unmodified full KV cache (Section 4.3): the T new tokens are
 * checked in one parallel pass.  q [device] bf16 [batch][T][Hq][D]; row j attends causally to cache
 * entries [0, kv_len[b] - T + j] (its own K/V is already in the cache).  Outputs as in draft_attend.
 * T * (Hq/Hkv) must be <= 64. */
int verify_attend(const masw_kv_desc* kv, const void* q, int T, float* o, float* lse, void* o_bf16,
                  void* workspace /*[device]*/, size_t workspace_bytes, void* stream);

/* A paged verifier cache (the serving layout for heterogeneous batches, Section 5.1): a pool of pages of
 * 128 entries, K and V laid out [page][kv head][128][head_dim] bf16, and a page table per sequence. */
typedef struct masw_paged_kv_desc {
  const void* k_pages;       /* [device] bf16 [n_pages][n_kv_heads][128][head_dim] */
  const void* v_pages;       /* [device] bf16, same layout */
  const int32_t* page_table; /* [device] [batch][max_pages]: pool page holding entries [128 i, 128 i + 128) of the sequence */
  int32_t n_pages, max_pages;
  int32_t batch, n_q_heads, n_kv_heads, head_dim; /* head_dim must be 128 */
  const int32_t* kv_len;     /* [device] [batch] entries in use, INCLUDING the T rows being verified; <= 128 max_pages */
  float softmax_scale;       /* 0 selects 1 / sqrt(D) */
  int32_t flags;             /* MASW_KV_* bits, 0 for the defaults */
  int32_t* status;           /* [device] one int32 that receives MASW_STATUS_* bits (OR-ed in), or NULL */
} masw_paged_kv_desc;

/* Scratch bytes for verify_attend_paged (same rules as verify_workspace_bytes).  Host only. */
size_t verify_paged_workspace_bytes(const masw_paged_kv_desc* kv, int T);

/* verify_attend (Section 4.3) over a paged cache: identical results, the entries of sequence b being
 * gathered through page_table[b].  Table entries of pages a sequence does not use are never dereferenced
 * for data that counts (a tile beyond kv_len is masked), but should be valid page numbers or -1. */
int verify_attend_paged(const masw_paged_kv_desc* kv, const void* q, int T, float* o, float* lse, void* o_bf16,
                        void* workspace /*[device]*/, size_t workspace_bytes, void* stream);

/* An FP8 verifier cache (a serving variant beside the paged bf16 cache, Section 5.1: the target's KV bytes are what
 * Eq. 2's beta L d term counts, and e4m3 halves them).  Pages of 128 entries, K and V laid out
 * [page][kv head][128][head_dim] with ONE BYTE per element (e4m3: 1 sign, 4 exponent, 3 mantissa bits, bias 7, no
 * infinities), and one fp32 scale per (page, kv head) for K and for V.  The value an element stands for is
 * DEFINED as  fp16( e4m3_value x fp16(scale) )  (both roundings to nearest): the kernel forms exactly that product
 * when it turns a page into an fp16 operand tile, and attention is then exact arithmetic on those values (q is
 * rounded from bf16 to fp16 as well; probabilities go to the tensor cores as fp16). */
typedef struct masw_fp8_kv_desc {
  const void* k_pages;       /* [device] e4m3 bytes [n_pages][n_kv_heads][128][head_dim] */
  const void* v_pages;       /* [device] same layout */
  const float* k_scale;      /* [device] fp32 [n_pages][n_kv_heads] */
  const float* v_scale;      /* [device] fp32 [n_pages][n_kv_heads] */
  const int32_t* page_table; /* [device] [batch][max_pages]: pool page holding entries [128 i, 128 i + 128) of the sequence */
  int32_t n_pages, max_pages;
  int32_t batch, n_q_heads, n_kv_heads, head_dim; /* head_dim must be 128 */
  const int32_t* kv_len;     /* [device] [batch] entries in use, INCLUDING the T rows being verified; <= 128 max_pages */
  float softmax_scale;       /* 0 selects 1 / sqrt(D) */
  int32_t flags;             /* MASW_KV_DETERMINISTIC or 0 */
  int32_t* status;           /* [device] one int32 that receives MASW_STATUS_* bits (OR-ed in), or NULL */
} masw_fp8_kv_desc;

/* Scratch bytes for verify_attend_fp8 (same rules as verify_workspace_bytes).  Host only. */
size_t verify_fp8_workspace_bytes(const masw_fp8_kv_desc* kv, int T);

/* verify_attend (Section 4.3) over the FP8 paged cache: row j of the T new tokens attends causally to entries
 * [0, kv_len[b] - T + j], each standing for its dequantised value as defined above.  q [device] bf16
 * [batch][T][Hq][D]; outputs as in verify_attend.  T * (Hq/Hkv) must be <= 32. */
int verify_attend_fp8(const masw_fp8_kv_desc* kv, const void* q, int T, float* o, float* lse, void* o_bf16,
                      void* workspace /*[device]*/, size_t workspace_bytes, void* stream);

/* Bytes of scratch accept_reject needs.  Host only.  Zero-fill once before first use. */
size_t accept_workspace_bytes(int batch, int gamma, int vocab);

/* The standard speculative-sampling accept/reject rule (Section 3.1; Section 4.3).
 * target_logits [device] bf16 [batch][gamma+1][V]; draft_logits [device] bf16 [batch][gamma][V] (may
 * be NULL when temperature == 0); draft_tokens [device] int32 [batch][gamma]; uniforms [device] fp32
 * [batch][gamma+1] in [0,1) (unused when temperature == 0).
 * temperature == 0 (the paper's evaluated mode): n = number of leading draft tokens equal to the
 *   arg-max of the target row (ties: lowest index); out_tokens = those n tokens followed by the
 *   arg-max of target row n (a correction if n < gamma, the bonus token if n == gamma).
 * temperature > 0: token i is accepted iff u_i * q_i(x_i) < p_i(x_i); at the first rejection the
 *   replacement is drawn from norm(max(0, p_n - q_n)); with no rejection the bonus is drawn from
 *   p_gamma; the final draw always uses uniforms[b][gamma].  Probabilities are 40-bit fixed-point
 *   integer weights and all comparisons are exact integer arithmetic, so decisions are reproducible
 *   bit for bit on any conforming implementation.  The sums of those weights are kept in 64 bits, which
 *   holds for vocab <= 131071 (the worst case, p and q flat on disjoint halves of the vocabulary, sums to
 *   vocab^2 2^30): a larger vocabulary is refused with MASW_EINVAL when temperature > 0.
 * Outputs: n_accepted [device] int32 [batch]; out_tokens [device] int32 [batch][gamma+1], unused = -1;
 * status [device] int32 or NULL receives MASW_STATUS_BAD_* bits (OR-ed in). */
int accept_reject(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                  const float* uniforms, int batch, int gamma, int vocab, float temperature,
                  int32_t* n_accepted, int32_t* out_tokens, int32_t* status,
                  void* workspace /*[device]*/, size_t workspace_bytes, void* stream);

/* Same rule and same outputs as accept_reject, for callers that cannot allocate device memory at the
 * point where they decide on the drafted tokens: a serving loop that has handed all of its device
 * memory to its own pool at start-up, or code that runs where cudaMalloc is off limits because it
 * would stall the device (it synchronises) in the middle of latency-critical decoding.  (The paper has
 * no counterpart: this is a convenience of this library.)  The scratch that accept_reject takes from
 * the caller lives here in a fixed array inside the library's device image (about 43 KB, present on
 * every GPU that loads the library until the process exits), so this call neither takes a workspace
 * nor calls cudaMalloc, cudaFree or any allocating routine.
 * Limits: batch <= 64 and gamma <= 16; larger requests fail with MASW_ECAPACITY and nothing is launched.
 * The first call on each device looks up the array's device address (once, with that device
 * current); make that first call before any stream capture begins.
 * All calls on a device share the one array and each call overwrites what the previous one left (the
 * part that must start at zero is cleared on `stream` first): calls that overlap on the GPU race, so
 * order them on one stream or with events. */
int accept_reject_static(const void* target_logits, const void* draft_logits, const int32_t* draft_tokens,
                         const float* uniforms, int batch, int gamma, int vocab, float temperature,
                         int32_t* n_accepted, int32_t* out_tokens, int32_t* status, void* stream);

/* Text of the most recent error on this thread ("" if none). */
const char* masw_last_error(void);

/* Number of kernels this library has launched in this process (for benchmarks' launch accounting). */
uint64_t masw_launch_count(void);

/* Library version string. */
const char* masw_version(void);

#ifdef __cplusplus
}
#endif
#endif /* MASW_H_ */
