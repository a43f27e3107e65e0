"""GPU parity: the draft's masked prefill pass (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from oracle import prefill as opf
from paper_2608_30252_b200 import binding, inputs
from helpers import assert_attention_close, dev_bf16, f64, host_bits

pytestmark = pytest.mark.gpu


LSE_TOL = 2e-3


def _mem(B, Hq, Hkv, D, S, W, r, max_slots, L=1):
    gamma_max = min(4, 64 // (Hq // Hkv) - 1)   # the decoding side packs (gamma_max + 1) x group rows into one tile
    cfg = binding.MaswConfig(L, B, Hq, Hkv, D, Hq * D, S, W, r, rollback=16, max_slots=max_slots, gamma_max=gamma_max)
    return binding.DraftMemory(cfg)


def _inputs(rng, B, Hq, Hkv, D, P, M, q_scale=1.0):
    qb = inputs.normal_bf16(rng, (B, P + M, Hq, D), std=q_scale)
    kb = inputs.normal_bf16(rng, (B, Hkv, P + M, D))
    vb = inputs.normal_bf16(rng, (B, Hkv, P + M, D))
    return qb, kb, vb


def _oracle(qb, kb, vb, P, S, W, r, rows=None):
    """Full oracle pass, or only the listed rows (index into the P + M rows) when `rows` is given."""
    q, k, v = f64(qb), f64(kb).transpose(0, 2, 1, 3), f64(vb).transpose(0, 2, 1, 3)   # k, v -> [B, n, Hkv, D]
    if rows is None:
        o_raw, l_raw, o_slot, l_slot = opf.prefill_attend(q[:, :P], q[:, P:], k[:, :P], v[:, :P], k[:, P:], v[:, P:], S, W, r)
        return np.concatenate([o_raw, o_slot], axis=1), np.concatenate([l_raw, l_slot], axis=1)
    B, _, Hq, D = q.shape
    G = Hq // k.shape[2]
    o, lse = np.zeros((B, len(rows), Hq, D)), np.zeros((B, len(rows), Hq))
    for b in range(B):
        for n, row in enumerate(rows):
            sink, n_slots, local = opf.raw_row_view(row, S, W, r) if row < P else opf.slot_row_view(row - P + 1, S, W, r)
            idx = list(sink) + [P + j for j in range(n_slots)] + list(local)
            for h in range(Hq):
                o[b, n, h], lse[b, n, h], _ = oracle.attend(q[b, row, h], k[b, idx, h // G], v[b, idx, h // G], D ** -0.5)
    return o, lse


def _case(rng, B, Hq, Hkv, D, S, W, r, P, q_scale=1.0, strided=False):
    M = opf.n_prefill_slots(P, S, r)
    g = _mem(B, Hq, Hkv, D, S, W, r, max(M, 1))
    assert g.draft_prefill_slots(P) == M
    qb, kb, vb = _inputs(rng, B, Hq, Hkv, D, P, M, q_scale)
    if strided:   # stored [B, n, Hkv, D], viewed as [B, Hkv, n, D]
        k = dev_bf16(np.ascontiguousarray(kb.transpose(0, 2, 1, 3))).permute(0, 2, 1, 3)
        v = dev_bf16(np.ascontiguousarray(vb.transpose(0, 2, 1, 3))).permute(0, 2, 1, 3)
    else:
        k, v = dev_bf16(kb), dev_bf16(vb)
    o_bf = torch.empty((B, P + M, Hq, D), dtype=torch.bfloat16, device="cuda")
    og, lg, _ = g.draft_prefill_attend(0, k, v, dev_bf16(qb), P, out_bf16=o_bf)
    _, _, status = g.mem_get_state()
    assert status == 0
    oref, lref = _oracle(qb, kb, vb, P, S, W, r)
    tag = f"prefill B{B} Hq{Hq}/{Hkv} D{D} S{S} W{W} r{r} P{P}"
    res = assert_attention_close(og.cpu().numpy(), oref, lg.cpu().numpy(), lref, tag=tag, lse_tol=LSE_TOL)
    # the optional bf16 output is the rounded fp32 output
    assert torch.equal(o_bf, og.to(torch.bfloat16))
    g.close()
    return res


@pytest.mark.parametrize("D", [64, 128])
def test_several_row_tiles_ragged_tails_sinks_slots_and_window(D):
    """G = 4: 32 tokens per query tile; prefix lengths that end inside a tile; windows shorter and longer than a
    KV tile; slot tiles with a ragged tail."""
    rng = inputs.rng_for(1, 0, 70 + D)
    _case(rng, 1, 8, 2, D, 5, 70, 4, 300)
    _case(rng, 2, 8, 2, D, 0, 200, 8, 333)
    _case(rng, 1, 4, 1, D, 130, 40, 3, 257)


@pytest.mark.parametrize("G", [1, 2, 8, 16])
def test_group_sizes(G):
    rng = inputs.rng_for(1, 0, 80 + G)
    _case(rng, 1, 2 * G, 2, 64, 3, 50, 5, 190)


def test_degenerate_prefixes():
    rng = inputs.rng_for(1, 0, 90)
    _case(rng, 1, 8, 2, 64, 8, 16, 4, 1)          # a single token
    _case(rng, 1, 8, 2, 64, 8, 16, 4, 6)          # shorter than the sink region
    _case(rng, 1, 8, 2, 64, 8, 16, 4, 8)          # exactly the sinks: no slot yet
    _case(rng, 1, 8, 2, 64, 0, 500, 1000, 140)    # no slots, window longer than the prefix: plain causal
    _case(rng, 1, 8, 2, 64, 0, 1, 1, 70)          # a slot after every token, window of one
    _case(rng, 1, 8, 2, 64, 4, 32, 4, 4 + 4 * 32) # slot count a multiple of the query tile


def test_peaky_scores_and_strided_cache():
    rng = inputs.rng_for(1, 0, 91)
    _case(rng, 1, 8, 2, 64, 2, 100, 4, 260, q_scale=6.0)
    _case(rng, 2, 8, 2, 128, 2, 100, 4, 260, strided=True)


def test_prefill_builds_the_memory_decoding_continues_from():
    """import_memory: after the pass and mem_set_state the draft attends exactly to what token-by-token
    decoding would have built (checked against the decoding oracle)."""
    rng = inputs.rng_for(1, 0, 92)
    B, Hq, Hkv, D, S, W, r, P = 2, 8, 2, 64, 4, 48, 4, 230
    M = opf.n_prefill_slots(P, S, r)
    g = _mem(B, Hq, Hkv, D, S, W, r, M + 8)
    qb, kb, vb = _inputs(rng, B, Hq, Hkv, D, P, M)
    g.draft_prefill_attend(0, dev_bf16(kb), dev_bf16(vb), dev_bf16(qb), P, import_memory=True)
    g.mem_set_state([P] * B, [M] * B)
    o = oracle.DraftMemory(1, B, Hq, Hkv, D, S, W, r)
    kf, vf = f64(kb).transpose(0, 2, 1, 3), f64(vb).transpose(0, 2, 1, 3)
    o.append_raw(0, kf[:, :P], vf[:, :P])
    o.load_slots(0, kf[:, P:], vf[:, P:])
    o.t, o.M = [P] * B, [M] * B
    for step in range(6):   # a few decoding steps on top, crossing a boundary
        k1, v1 = inputs.normal_bf16(rng, (B, 1, Hkv, D)), inputs.normal_bf16(rng, (B, 1, Hkv, D))
        q1 = inputs.normal_bf16(rng, (B, 1, Hq, D))
        boundary = o.boundary_after(0)
        o.append_raw(0, f64(k1), f64(v1))
        oref, lref = o.attend(0, f64(q1))
        og, lg = g.draft_append_attend(0, dev_bf16(k1), dev_bf16(v1), dev_bf16(q1))
        assert_attention_close(og.cpu().numpy(), oref, lg.cpu().numpy(), lref, tag=f"decode after prefill, step {step}")
        if boundary:   # keep the two memories in step: install the same slot on both sides
            ks, vs = inputs.normal_bf16(rng, (B, 1, Hkv, D)), inputs.normal_bf16(rng, (B, 1, Hkv, D))
            o.load_slots(0, f64(ks), f64(vs))
            g.mem_load(0, binding.REGION_SLOT, dev_bf16(ks), dev_bf16(vs), first=o.M[0])
        o.advance(1, slot_added=[boundary] * B)
        g.mem_advance(1, add_slot=boundary)
    g.close()


@pytest.mark.parametrize("name", ["cfg3_8b_32k", "cfg4_70b_32k"])
def test_full_size_prefix_sampled_rows(name):
    """The 32K prefix of the benchmark's draft shapes (head_dim 64 and head_dim 128), one layer: sampled rows (first and last tokens, rows
    around tile and window edges, slot rows) against the oracle, row by row."""
    wl = inputs.WORKLOADS[name]
    rng = inputs.rng_for(3, 0, 93)
    B, Hq, Hkv, D = 1, wl.d_q_heads, wl.d_kv_heads, wl.d_head_dim
    S, W, r, P = wl.sink, wl.window, wl.slot_interval, wl.prefix
    M = opf.n_prefill_slots(P, S, r)
    g = _mem(B, Hq, Hkv, D, S, W, r, M)
    gen = torch.Generator(device="cuda").manual_seed(260830252)
    q = torch.randn((B, P + M, Hq, D), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    k = torch.randn((B, Hkv, P + M, D), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    v = torch.randn((B, Hkv, P + M, D), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    og, lg, _ = g.draft_prefill_attend(0, k, v, q, P)
    _, _, status = g.mem_get_state()
    assert status == 0
    rows = sorted(set([0, 1, 31, 32, 127, 128, W - 1, W, W + 1, 2 * W + 17, P // 2, P - 129, P - 2, P - 1,
                       P, P + 1, P + 31, P + 32, P + M // 2, P + M - 1] + [int(x) for x in rng.integers(0, P + M, 12)]))
    oref, lref = _oracle(host_bits(q), host_bits(k), host_bits(v), P, S, W, r, rows=rows)
    assert_attention_close(og[:, rows].cpu().numpy(), oref, lg[:, rows].cpu().numpy(), lref, tag=f"prefill {name}", lse_tol=LSE_TOL)
    g.close()
