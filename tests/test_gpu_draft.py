"""GPU parity: draft memory update + draft attention (through the C ABI) against the CPU oracle."""
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2608_30252_b200 import binding, inputs
from helpers import assert_attention_close, bf16_ulp_distance, dev_bf16, f64, host_bits

pytestmark = pytest.mark.gpu


class Pair:
    """A GPU draft memory and the oracle's, driven in lock-step with the same seeded inputs."""

    def __init__(self, rng, L, B, Hq, Hkv, D, S, W, r, max_slots, gamma_max=4, rollback=16, d_model=None):
        self.rng, self.L, self.B, self.Hq, self.Hkv, self.D = rng, L, B, Hq, Hkv, D
        self.d = d_model or Hq * D
        self.cfg = binding.MaswConfig(L, B, Hq, Hkv, D, self.d, S, W, r, rollback=rollback, max_slots=max_slots,
                                      gamma_max=gamma_max)
        self.g = binding.DraftMemory(self.cfg)
        self.o = oracle.DraftMemory(L, B, Hq, Hkv, D, S, W, r)
        self.Wk = [inputs.normal_bf16(rng, (self.d, Hkv * D), self.d ** -0.5) for _ in range(L)]
        self.Wv = [inputs.normal_bf16(rng, (self.d, Hkv * D), self.d ** -0.5) for _ in range(L)]
        self.dWk = [dev_bf16(w) for w in self.Wk]
        self.dWv = [dev_bf16(w) for w in self.Wv]
        self.worst = (0.0, 0.0)
        self.slot_ulps = 0
        self.deferred = False   # counter updates noted on the host only (mem_advance_deferred)

    def step(self, n_raw=1, check=True, q_scale=1.0, fused=False, fused_slot=False):
        o, rng = self.o, self.rng
        boundary = [o.boundary_after(b, n_raw) for b in range(self.B)]
        fire = any(boundary)
        act = torch.tensor(boundary, dtype=torch.uint8, device="cuda")
        for l in range(self.L):
            k = inputs.normal_bf16(rng, (self.B, n_raw, self.Hkv, self.D))
            v = inputs.normal_bf16(rng, (self.B, n_raw, self.Hkv, self.D))
            o.append_raw(l, f64(k), f64(v))
            if not fused:
                self.g.mem_update(l, k_raw=dev_bf16(k), v_raw=dev_bf16(v))
            one_launch = fire and fused and fused_slot
            if fire:
                h = inputs.normal_bf16(rng, (self.B, self.d))
                pos = [o.t[b] + n_raw for b in range(self.B)]
                Ko, Vo = o.materialize(l, f64(h), f64(self.Wk[l]), f64(self.Wv[l]), pos, active=boundary)
                dpos = torch.tensor(pos, dtype=torch.int32, device="cuda")
                if not one_launch:
                    self.g.mem_update(l, h_g=dev_bf16(h), Wk_g=self.dWk[l], Wv_g=self.dWv[l], slot_pos=dpos, active=act)
                if check and not one_launch:
                    Kg, Vg = self.g.kv_view(l)
                    for b in range(self.B):
                        if not boundary[b]:
                            continue
                        e = self.cfg.sink + o.M[b]
                        # stored slot K/V: the oracle's bf16 value or its neighbour (fp32 vs fp64
                        # accumulation may flip a rounding; where RoPE cancels to ~0 an absolute floor applies)
                        for got, ref in ((host_bits(Kg[b, :, e]), Ko[b]), (host_bits(Vg[b, :, e]), Vo[b])):
                            diff = np.abs(f64(got) - ref)
                            assert (diff <= 2.0 ** -7 * np.abs(ref) + 1e-5).all(), diff.max()
                            flips = bf16_ulp_distance(got, oracle.f64_to_bf16_bits(ref)) > 0
                            assert flips.mean() < 0.05
                            self.slot_ulps += int(flips.sum())
            n_q = n_raw + (1 if fire else 0)
            q = inputs.normal_bf16(rng, (self.B, n_q, self.Hq, self.D), std=q_scale)
            if one_launch:
                og, lg = self.g.draft_boundary_attend(l, dev_bf16(k), dev_bf16(v), dev_bf16(h), self.dWk[l], self.dWv[l],
                                                      dpos, dev_bf16(q), active=act)
                if check:
                    Kg, Vg = self.g.kv_view(l)
                    for b in range(self.B):
                        if not boundary[b]:
                            continue
                        e = self.cfg.sink + o.M[b]
                        for got, ref in ((host_bits(Kg[b, :, e]), Ko[b]), (host_bits(Vg[b, :, e]), Vo[b])):
                            diff = np.abs(f64(got) - ref)
                            assert (diff <= 2.0 ** -7 * np.abs(ref) + 1e-5).all(), diff.max()
            elif fused:
                og, lg = self.g.draft_append_attend(l, dev_bf16(k), dev_bf16(v), dev_bf16(q), last_row_is_slot=fire)
            else:
                og, lg = self.g.draft_attend(l, dev_bf16(q), last_row_is_slot=fire)
            if check:
                oref, lref = o.attend(l, f64(q), last_row_is_slot=fire, active=boundary)
                mx, rel = assert_attention_close(og.cpu().numpy(), oref, lg.cpu().numpy(), lref, tag=f"t={o.t} l={l}")
                self.worst = (max(self.worst[0], mx), max(self.worst[1], rel))
        o.advance(n_raw, slot_added=boundary)
        if self.deferred:
            assert all(boundary) == any(boundary)   # a deferred update has no per-sequence mask
            self.g.mem_advance(n_raw, add_slot=fire, deferred=True)
        else:
            self.g.mem_advance(n_raw, add_slot=fire, active=act)

    def check_state(self):
        t, m, status = self.g.mem_get_state()
        assert t == self.o.t and m == self.o.M and status == 0, (t, m, status, self.o.t, self.o.M)


def test_cfg1_stream_1024_tokens_every_step():
    """Config 1 draft side: 8 q / 2 KV heads, D = 64, r = 16, W = 64, memory built token by token by
    the adaptor with random-init weights over a 1024-token stream; every step's attention is checked."""
    p = Pair(inputs.rng_for(1, 0, 0), L=1, B=1, Hq=8, Hkv=2, D=64, S=0, W=64, r=16, max_slots=64)
    for _ in range(1024):
        p.step()
    p.check_state()
    assert p.o.M[0] == 64 and p.o.n_visible(0) == 128
    assert p.worst[1] < 2e-4, p.worst       # the single row block carries p as hi + lo bf16 terms


def test_paper_constants_scaled_down_with_sinks_ring_wrap_layers_and_ragged_batch():
    """Sink filling from t = 0, ring wrap-around (the ring is 64 entries), two layers, two sequences
    whose boundaries fire on different steps (per-sequence `active`)."""
    p = Pair(inputs.rng_for(6, 0, 1), L=2, B=2, Hq=4, Hkv=2, D=64, S=5, W=12, r=4, max_slots=80, rollback=4)
    # de-synchronise the two sequences: sequence 1 starts two tokens ahead
    p.o.t[1] = 2
    for l in range(2):
        p.o.raw[l][1] = [(np.zeros((2, 64)), np.zeros((2, 64)))] * 2
    p.g.mem_set_state(t=[0, 2], n_slots=[0, 0])
    for _ in range(150):
        p.step()
    p.check_state()
    assert p.o.M[0] != p.o.M[1] or p.o.t[0] != p.o.t[1]


def test_fused_append_attend_matches_the_two_call_sequence():
    """draft_append_attend == mem_update(raw) + draft_attend: sinks filling from t = 0, ring wrap, slot rows,
    two layers, ragged batch; later steps read the appended tokens back from the arena."""
    p = Pair(inputs.rng_for(6, 0, 9), L=2, B=2, Hq=8, Hkv=2, D=64, S=5, W=12, r=4, max_slots=80, rollback=4)
    p.o.t[1] = 2
    for l in range(2):
        p.o.raw[l][1] = [(np.zeros((2, 64)), np.zeros((2, 64)))] * 2
    p.g.mem_set_state(t=[0, 2], n_slots=[0, 0])
    for _ in range(150):
        p.step(fused=True)
    p.check_state()
    q = Pair(inputs.rng_for(6, 0, 10), L=1, B=1, Hq=8, Hkv=2, D=128, S=3, W=70, r=5, max_slots=64, gamma_max=3, rollback=4,
             d_model=256)
    for i in range(60):
        q.step(n_raw=3 if i % 2 else 1, fused=(i % 3 != 0))      # mixed fused / unfused, multi-token rows
    q.check_state()


@pytest.mark.parametrize("D,Hq,Hkv,n_raw", [(64, 8, 2, 7), (64, 8, 1, 5), (64, 16, 2, 7), (128, 8, 2, 7), (128, 8, 1, 5), (128, 16, 2, 7)])
def test_wide_query_tiles_two_to_four_row_blocks(D, Hq, Hkv, n_raw):
    """Many pending rows per call: (n_raw + slot row) x group heads = 32 .. 64 query rows, i.e. two to four
    16-row blocks of the mma.sync kernel, for both head dims, fused and unfused append."""
    p = Pair(inputs.rng_for(6, 0, 11 + D + Hq + n_raw), L=1, B=1, Hq=Hq, Hkv=Hkv, D=D, S=3, W=40, r=n_raw, max_slots=64,
             gamma_max=n_raw, rollback=4, d_model=256)
    for i in range(12):
        p.step(n_raw=n_raw, fused=bool(i % 2))
    p.check_state()


def test_boundary_step_in_one_launch():
    """draft_boundary_attend == mem_update(raw) + mem_update(slot) + draft_attend(slot row): both head dims,
    ragged batch with per-sequence `active`, ring wrap, two layers, multi-token rows; the stored slot is
    read back and later steps attend over it."""
    p = Pair(inputs.rng_for(6, 0, 12), L=2, B=2, Hq=8, Hkv=2, D=64, S=5, W=12, r=4, max_slots=80, rollback=4)
    p.o.t[1] = 2
    for l in range(2):
        p.o.raw[l][1] = [(np.zeros((2, 64)), np.zeros((2, 64)))] * 2
    p.g.mem_set_state(t=[0, 2], n_slots=[0, 0])
    for _ in range(120):
        p.step(fused=True, fused_slot=True)
    p.check_state()
    q = Pair(inputs.rng_for(6, 0, 13), L=1, B=1, Hq=8, Hkv=2, D=128, S=3, W=70, r=6, max_slots=64, gamma_max=3, rollback=4,
             d_model=256)
    for i in range(40):
        q.step(n_raw=3, fused=True, fused_slot=(i % 4 != 0))
    q.check_state()


@pytest.mark.parametrize("D", [64, 128])
def test_every_instance_of_the_decode_kernel(D):
    """The decode kernel is compiled per (head_dim, packed probability terms or not, slot materialisation or not).
    Groups of one, two and four heads with one to three pending tokens put one to eight rows on a KV head, so that
    every instance runs: rows of different tokens (different visibility bounds) inside the packed instance, the
    packed instance with the fused slot (group of two: raw row + slot row = four rows), the unpacked ones beside
    them; ragged batch, sinks, ring wrap, the stored slot read back and attended over by later steps."""
    seed = 40 + D
    for Hq, Hkv, n_raw, steps in ((2, 2, 1, 60), (2, 2, 3, 30), (4, 2, 1, 80), (4, 2, 2, 40), (4, 2, 3, 30), (8, 2, 1, 60)):
        p = Pair(inputs.rng_for(6, 0, seed), L=1, B=2, Hq=Hq, Hkv=Hkv, D=D, S=3, W=20, r=2 * n_raw, max_slots=96, gamma_max=3,
                 rollback=4, d_model=128)
        seed += 1
        p.o.t[1] = n_raw
        p.o.raw[0][1] = [(np.zeros((Hkv, D)), np.zeros((Hkv, D)))] * n_raw
        p.g.mem_set_state(t=[0, n_raw], n_slots=[0, 0])
        for i in range(steps):
            p.step(n_raw=n_raw, fused=True, fused_slot=(i % 3 != 0))
        p.check_state()
        assert p.worst[1] < 1e-4, (Hq, Hkv, n_raw, p.worst)   # both bf16 terms of the probabilities are in the result


def test_multi_token_pending_rows_and_slot_row():
    """n_raw > 1 pending tokens per call (causal among themselves) with the slot row riding on the last."""
    p = Pair(inputs.rng_for(6, 0, 2), L=1, B=1, Hq=8, Hkv=2, D=64, S=3, W=10, r=3, max_slots=64, gamma_max=3, rollback=4)
    for _ in range(30):
        p.step(n_raw=3)
    p.check_state()


def test_head_dim_128_group_of_four():
    p = Pair(inputs.rng_for(4, 0, 3), L=1, B=2, Hq=8, Hkv=2, D=128, S=2, W=40, r=8, max_slots=32, d_model=256)
    for _ in range(100):
        p.step()
    p.check_state()


def test_peaky_scores_where_max_abs_bites():
    """Queries scaled x6: a few keys dominate and the outputs are O(1), so the absolute bound matters."""
    p = Pair(inputs.rng_for(1, 0, 4), L=1, B=1, Hq=8, Hkv=2, D=64, S=0, W=64, r=16, max_slots=64)
    for i in range(200):
        p.step(q_scale=6.0)


def _loaded_case(wl, layer_count, layer, rng, fused=False):
    """Memory filled directly (prefill import): M slots + W window tokens, one decode step on top."""
    B, Hq, Hkv, D, S, M, W = wl.batch, wl.d_q_heads, wl.d_kv_heads, wl.d_head_dim, wl.sink, wl.slots, wl.window
    cfg = binding.MaswConfig(layer_count, B, Hq, Hkv, D, wl.d_model, S, W, wl.slot_interval, rollback=16,
                             max_slots=M + 8, gamma_max=8)
    g = binding.DraftMemory(cfg)
    t0 = S + M * wl.slot_interval            # tokens committed so far
    ks, vs = inputs.normal_bf16(rng, (B, M, Hkv, D)), inputs.normal_bf16(rng, (B, M, Hkv, D))
    kw, vw = inputs.normal_bf16(rng, (B, W, Hkv, D)), inputs.normal_bf16(rng, (B, W, Hkv, D))
    g.mem_load(layer, binding.REGION_SLOT, dev_bf16(ks), dev_bf16(vs), first=0)
    g.mem_load(layer, binding.REGION_LOCAL, dev_bf16(kw), dev_bf16(vw), first=t0 - W)
    if S:
        ksk, vsk = inputs.normal_bf16(rng, (B, S, Hkv, D)), inputs.normal_bf16(rng, (B, S, Hkv, D))
        g.mem_load(layer, binding.REGION_SINK, dev_bf16(ksk), dev_bf16(vsk), first=0)
    g.mem_set_state(t=[t0] * B, n_slots=[M] * B)
    kn, vn = inputs.normal_bf16(rng, (B, 1, Hkv, D)), inputs.normal_bf16(rng, (B, 1, Hkv, D))
    q = inputs.normal_bf16(rng, (B, 1, Hq, D))
    # The first launch follows a counter update and reads everything behind its wait; the launches after it
    # follow an attention launch and may run ahead of it (plan and K/V copies before the wait, the CTA's first
    # tile kept in registers).  The two orders sum the same entries in a different order, so each is checked
    # against the oracle, and the repeated order must give the same bits (run-to-run determinism).
    if fused:      # the launch the benchmark times: append fused into the attention
        call = lambda: g.draft_append_attend(layer, dev_bf16(kn), dev_bf16(vn), dev_bf16(q))
    else:
        g.mem_update(layer, k_raw=dev_bf16(kn), v_raw=dev_bf16(vn))
        call = lambda: g.draft_attend(layer, dev_bf16(q))
    (og, lg), (og2, lg2), (og3, lg3) = call(), call(), call()
    assert torch.equal(og2, og3) and torch.equal(lg2, lg3)
    g.mem_advance(0)                                              # a counter update: the next launch waits first again
    og4, lg4 = call()
    assert torch.equal(og, og4) and torch.equal(lg, lg4)
    # oracle: the plain definition over the explicit entry list
    G = Hq // Hkv
    scale = 1 / math.sqrt(D)
    oref = np.zeros((B, 1, Hq, D)); lref = np.zeros((B, 1, Hq))
    for b in range(B):
        parts_k = [f64(ks[b]), f64(kw[b, 1:]), f64(kn[b])]        # the oldest window token just left
        parts_v = [f64(vs[b]), f64(vw[b, 1:]), f64(vn[b])]
        if S:
            parts_k.insert(0, f64(ksk[b])); parts_v.insert(0, f64(vsk[b]))
        K = np.concatenate(parts_k); V = np.concatenate(parts_v)
        assert len(K) == S + M + W
        for h in range(Hq):
            oref[b, 0, h], lref[b, 0, h], _ = oracle.attend(f64(q[b, 0, h]), K[:, h // G], V[:, h // G], scale)
    assert_attention_close(og2.cpu().numpy(), oref, lg2.cpu().numpy(), lref, tag=wl.name + " (ahead of its predecessor)", rel_tol=2e-4)
    mx, rel = assert_attention_close(og.cpu().numpy(), oref, lg.cpu().numpy(), lref, tag=wl.name, rel_tol=2e-4)
    assert g.mem_get_state()[2] == 0
    return mx, rel


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("name", ["cfg2_8b_8k", "cfg3_8b_32k", "cfg4_70b_32k", "paper_r4_32k", "paper_r8_32k"])
def test_full_size_memory_in_bench_launch_configuration(name, fused):
    """Full-size draft memories (the benchmark's shapes), all heads of one layer checked element by
    element; the layer index is not 0 so that per-layer arena offsets are exercised.  `fused` is the
    launch the benchmark times (draft_append_attend)."""
    wl = inputs.WORKLOADS[name]
    _loaded_case(wl, layer_count=3, layer=2, rng=inputs.rng_for(wl.config_id, 2, 5), fused=fused)


@pytest.mark.parametrize("name", ["cfg3_8b_32k", "cfg4_70b_32k"])
def test_full_size_boundary_launches_ahead_of_their_predecessor(name):
    """The benchmark's boundary launch at full size: draft_boundary_attend on consecutive layers, so that every launch
    but the first runs ahead of its predecessor (plan, K/V copies, first tile in registers and the projection's weight
    rows before the wait; 18 k-splits of the slot projection).  Each layer's two rows and its stored slot are checked
    against the oracle."""
    wl = inputs.WORKLOADS[name]
    rng = inputs.rng_for(wl.config_id, 3, 6)
    B, Hq, Hkv, D, S, M, W = wl.batch, wl.d_q_heads, wl.d_kv_heads, wl.d_head_dim, wl.sink, wl.slots, wl.window
    L, d = 3, wl.d_model
    cfg = binding.MaswConfig(L, B, Hq, Hkv, D, d, S, W, wl.slot_interval, rollback=16, max_slots=M + 8, gamma_max=8)
    g = binding.DraftMemory(cfg)
    t0 = S + M * wl.slot_interval
    data = []
    for l in range(L):
        ks, vs = inputs.normal_bf16(rng, (B, M, Hkv, D)), inputs.normal_bf16(rng, (B, M, Hkv, D))
        kw, vw = inputs.normal_bf16(rng, (B, W, Hkv, D)), inputs.normal_bf16(rng, (B, W, Hkv, D))
        g.mem_load(l, binding.REGION_SLOT, dev_bf16(ks), dev_bf16(vs), first=0)
        g.mem_load(l, binding.REGION_LOCAL, dev_bf16(kw), dev_bf16(vw), first=t0 - W)
        kn, vn = inputs.normal_bf16(rng, (B, 1, Hkv, D)), inputs.normal_bf16(rng, (B, 1, Hkv, D))
        h = inputs.normal_bf16(rng, (B, d))
        Wk, Wv = inputs.normal_bf16(rng, (d, Hkv * D), d ** -0.5), inputs.normal_bf16(rng, (d, Hkv * D), d ** -0.5)
        q = inputs.normal_bf16(rng, (B, 2, Hq, D))
        data.append((ks, vs, kw, vw, kn, vn, h, Wk, Wv, q))
    g.mem_set_state(t=[t0] * B, n_slots=[M] * B)
    pos = torch.tensor([t0 + 1] * B, dtype=torch.int32, device="cuda")
    dev = [[dev_bf16(x) for x in (kn, vn, h, Wk, Wv, q)] for (_, _, _, _, kn, vn, h, Wk, Wv, q) in data]
    outs = [g.draft_boundary_attend(l, dev[l][0], dev[l][1], dev[l][2], dev[l][3], dev[l][4], pos, dev[l][5]) for l in range(L)]
    torch.cuda.synchronize()
    assert g.mem_get_state()[2] == 0
    G, scale = Hq // Hkv, 1 / math.sqrt(D)
    o = oracle.DraftMemory(1, B, Hq, Hkv, D, S, W, wl.slot_interval)
    for l, (ks, vs, kw, vw, kn, vn, h, Wk, Wv, q) in enumerate(data):
        Ko, Vo = o.materialize(0, f64(h), f64(Wk), f64(Wv), [t0 + 1] * B)
        Kg, Vg = g.kv_view(l)
        og, lg = outs[l]
        for b in range(B):
            for got, ref in ((host_bits(Kg[b, :, S + M]), Ko[b]), (host_bits(Vg[b, :, S + M]), Vo[b])):
                assert (np.abs(f64(got) - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-5).all()
            # raw row: slots + window (oldest token left) + the new token; slot row: the same + the slot as stored
            Kr = np.concatenate([f64(ks[b]), f64(kw[b, 1:]), f64(kn[b])]); Vr = np.concatenate([f64(vs[b]), f64(vw[b, 1:]), f64(vn[b])])
            Ksl = np.concatenate([Kr, f64(host_bits(Kg[b, :, S + M]))[None]]); Vsl = np.concatenate([Vr, f64(host_bits(Vg[b, :, S + M]))[None]])
            oref = np.zeros((2, Hq, D)); lref = np.zeros((2, Hq))
            for hd in range(Hq):
                oref[0, hd], lref[0, hd], _ = oracle.attend(f64(q[b, 0, hd]), Kr[:, hd // G], Vr[:, hd // G], scale)
                oref[1, hd], lref[1, hd], _ = oracle.attend(f64(q[b, 1, hd]), Ksl[:, hd // G], Vsl[:, hd // G], scale)
            assert_attention_close(og[b].cpu().numpy(), oref, lg[b].cpu().numpy(), lref, tag=f"{name} boundary layer {l}", rel_tol=2e-4)
    g.close()


def test_sweep_shapes_batch_and_ratio():
    """A slice of the sweep grid: batch 4 and 16, memory ratio 10 % and 50 %."""
    for wl in inputs.sweep_workloads(prefixes=(4096,), batches=(4, 16), gammas=(5,), intervals=(20, 4)):
        _loaded_case(wl, layer_count=1, layer=0, rng=inputs.rng_for(5, 0, wl.batch * 100 + wl.slot_interval))


def test_empty_memory_and_first_token():
    """Degenerate cases: the very first token (one visible entry) and a memory with no slots."""
    p = Pair(inputs.rng_for(1, 0, 6), L=1, B=1, Hq=8, Hkv=2, D=64, S=0, W=8, r=10 ** 6, max_slots=0)
    for _ in range(20):
        p.step()
    p.check_state()
    assert p.o.M[0] == 0


def test_rollback_reexposes_window_and_drops_slots():
    p = Pair(inputs.rng_for(6, 0, 7), L=1, B=1, Hq=8, Hkv=2, D=64, S=2, W=8, r=3, max_slots=64, rollback=8)
    for _ in range(20):
        p.step()
    t_keep, m_keep = list(p.o.t), list(p.o.M)
    for _ in range(4):                      # speculative tokens, at least one slot among them
        p.step()
    assert p.o.M[0] > m_keep[0]
    p.o.rollback(t_keep, m_keep)
    p.g.mem_rollback(torch.tensor(t_keep, dtype=torch.int32, device="cuda"),
                     torch.tensor(m_keep, dtype=torch.int32, device="cuda"), slots_keep_max=max(m_keep))
    p.check_state()
    for _ in range(10):                     # decoding continues from the restored state
        p.step()
    p.check_state()


@pytest.mark.parametrize("D", [64, 128])
def test_deferred_counter_updates(D):
    """mem_advance_deferred notes the counter update on the host; the attention launches that follow and the
    rollback take it as launch parameters, every other call applies it first.  Speculative blocks of four draft
    steps (fused append, fused slot materialisation in the block) with nothing but attention launches between
    them, then a rollback that keeps 0..4 of the tokens (Section 4.3, "Rollback"); the counters are read back
    every other block (which applies what is pending), an unfused mem_update joins in now and then, and every
    attention output is checked against the oracle."""
    p = Pair(inputs.rng_for(6, 0, 70 + D), L=2, B=2, Hq=8, Hkv=2, D=D, S=3, W=24, r=4, max_slots=96, rollback=8, d_model=128)
    p.deferred = True
    for block in range(24):
        t_keep, m_keep = list(p.o.t), list(p.o.M)
        for j in range(4):
            p.step(fused=(block % 5 != 4), fused_slot=True)
        keep = block % 5
        if keep < 4:
            t_new = [t + keep for t in t_keep]
            m_new = [max(0, t - 3) // 4 for t in t_new]
            p.o.rollback(t_new, m_new)
            p.g.mem_rollback(torch.tensor(t_new, dtype=torch.int32, device="cuda"),
                             torch.tensor(m_new, dtype=torch.int32, device="cuda"), slots_keep_max=max(m_new))
        if block % 2 == 0:
            p.check_state()
    p.g.mem_flush()
    p.check_state()
    assert p.worst[1] < 2e-3


def test_slot_region_overflow_is_reported_not_written():
    p = Pair(inputs.rng_for(6, 0, 8), L=1, B=1, Hq=8, Hkv=2, D=64, S=0, W=8, r=2, max_slots=3)
    for _ in range(6):
        p.step()
    assert p.o.M[0] == 3
    with pytest.raises(binding.MaswError) as ei:
        p.step(check=False)
        p.step(check=False)
    assert ei.value.code == binding.MASW_ECAPACITY
