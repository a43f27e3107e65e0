"""GPU parity: the verifier's attention over its full KV cache against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_30252_b200 import binding, inputs
from helpers import assert_attention_close, dev_bf16, f64

pytestmark = pytest.mark.gpu


def _case(rng, B, Hq, Hkv, D, P, T, cap=None, lens=None, q_scale=1.0, poison=False, strided=False, rel_tol=2e-3):
    cap = cap or P + T
    lens = lens or [P + T] * B
    kb, vb = inputs.normal_bf16(rng, (B, Hkv, cap, D)), inputs.normal_bf16(rng, (B, Hkv, cap, D))
    qb = inputs.normal_bf16(rng, (B, T, Hq, D), std=q_scale)
    if strided:
        # cache stored [B, cap, Hkv, D] in memory and viewed as [B, Hkv, cap, D]
        k = dev_bf16(np.ascontiguousarray(kb.transpose(0, 2, 1, 3))).permute(0, 2, 1, 3)
        v = dev_bf16(np.ascontiguousarray(vb.transpose(0, 2, 1, 3))).permute(0, 2, 1, 3)
    else:
        k, v = dev_bf16(kb), dev_bf16(vb)
    if poison:
        for b in range(B):
            k[b, :, lens[b]:] = float("nan")
            v[b, :, lens[b]:] = float("nan")
    kv_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
    ws = binding.verify_workspace(k, kv_len, Hq, T)
    og, lg = binding.verify_attend(k, v, kv_len, dev_bf16(qb), workspace=ws)
    # the scratch is reusable; which split streams a pooled tile varies from launch to launch, and with it
    # each split's softmax reference and hence the bf16 rounding of its probabilities: a repeat agrees
    # within the parity tolerance, not bit for bit
    og2, lg2 = binding.verify_attend(k, v, kv_len, dev_bf16(qb), workspace=ws)
    d = (og - og2).double()
    assert float(d.pow(2).mean().sqrt()) <= 2 * rel_tol * float(og.double().pow(2).mean().sqrt()) + 1e-12   # two noisy runs
    assert torch.allclose(lg, lg2, rtol=1e-3, atol=1e-3)
    oref, lref = oracle.verify_attend(f64(qb), f64(kb), f64(vb), lens)
    # the deterministic mode (every tile assigned statically): same parity bar, and a repeat is bit-identical;
    # its status word stays clear
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    od, ld = binding.verify_attend(k, v, kv_len, dev_bf16(qb), workspace=ws, deterministic=True, status=status)
    od2, ld2 = binding.verify_attend(k, v, kv_len, dev_bf16(qb), workspace=ws, deterministic=True, status=status)
    assert torch.equal(od, od2) and torch.equal(ld, ld2), "deterministic verify_attend is not run-to-run identical"
    assert int(status.item()) == 0
    assert_attention_close(od.cpu().numpy(), oref, ld.cpu().numpy(), lref, tag=f"deterministic verify B{B} Hq{Hq} T{T} P{P}",
                           rel_tol=rel_tol)
    return assert_attention_close(og.cpu().numpy(), oref, lg.cpu().numpy(), lref, tag=f"verify B{B} Hq{Hq} T{T} P{P}", rel_tol=rel_tol)


def test_cfg1_target_gamma_and_gamma_plus_one_rows():
    """Config 1 target side: 8 q / 2 KV heads, D = 128, 1024-token cache, gamma = 4 (and gamma + 1 rows)."""
    rng = inputs.rng_for(1, 0, 10)
    _case(rng, 1, 8, 2, 128, 1024, 4)
    _case(rng, 1, 8, 2, 128, 1024, 5)


@pytest.mark.parametrize("T,G", [(1, 4), (5, 4), (6, 4), (6, 8), (7, 8), (8, 8), (3, 1), (2, 16)])
def test_row_block_counts_and_ragged_tails(T, G):
    """1 to 4 sixteen-row blocks; prefix lengths that end inside a tile."""
    rng = inputs.rng_for(4, 0, 11 + T * 10 + G)
    for P in (1, 63, 64, 65, 777, 2000):
        _case(rng, 1, 2 * G, 2, 128, P, T)


@pytest.mark.parametrize("T,G", [(4, 4), (5, 4), (6, 8), (8, 8), (3, 16)])
def test_head_dim_64_all_row_block_counts(T, G):
    """head_dim 64 runs on the mma.sync kernel: one to four 16-row blocks."""
    rng = inputs.rng_for(4, 0, 40 + T * 10 + G)
    for P in (5, 129, 1000):
        _case(rng, 1, 2 * G, 2, 64, P, T)


def test_degenerate_lengths():
    """Cache shorter than the row count (early rows see nothing and return zeros / -inf lse) and a single entry."""
    rng = inputs.rng_for(4, 0, 41)
    for D in (64, 128):
        kb, vb = inputs.normal_bf16(rng, (1, 2, 16, D)), inputs.normal_bf16(rng, (1, 2, 16, D))
        qb = inputs.normal_bf16(rng, (1, 4, 8, D))
        kv_len = torch.tensor([2], dtype=torch.int32, device="cuda")      # T = 4 rows, only 2 entries
        og, lg = binding.verify_attend(dev_bf16(kb), dev_bf16(vb), kv_len, dev_bf16(qb))
        og, lg = og.cpu().numpy(), lg.cpu().numpy()
        assert (og[0, :2] == 0).all() and np.isneginf(lg[0, :2]).all()   # rows 0, 1 see entries [0, -2], [0, -1]: nothing
        oref, lref = oracle.verify_attend(f64(qb)[:, 2:], f64(kb), f64(vb), [2])   # rows 2, 3 are a T = 2 problem
        assert_attention_close(og[:, 2:], oref, lg[:, 2:], lref, tag=f"short cache D{D}")


def test_batch_with_ragged_lengths_capacity_slack_and_poison_beyond_length():
    rng = inputs.rng_for(5, 0, 12)
    _case(rng, 3, 8, 2, 128, 500, 5, cap=640, lens=[505, 131, 640], poison=True)
    _case(rng, 2, 8, 2, 64, 300, 4, cap=512, lens=[304, 9], poison=True)


def test_strided_cache_view():
    rng = inputs.rng_for(5, 0, 13)
    _case(rng, 2, 8, 4, 128, 400, 5, strided=True)


def test_peaky_and_sink_like_scores():
    rng = inputs.rng_for(5, 0, 14)
    mx, _ = _case(rng, 1, 8, 2, 128, 4096, 5, q_scale=6.0)
    assert mx > 1e-5            # outputs are O(1) here, so the absolute bound is the one that bites


@pytest.mark.parametrize("name,T", [("cfg2_8b_8k", 5), ("cfg3_8b_32k", 5), ("cfg3_8b_32k", 6), ("cfg4_70b_32k", 6), ("cfg4_70b_32k", 7)])
def test_full_size_layer_in_bench_launch_configuration(name, T):
    """One full-size target layer (all heads, all rows) checked element by element."""
    wl = inputs.WORKLOADS[name]
    _case(inputs.rng_for(wl.config_id, 0, 15), wl.batch, wl.t_q_heads, wl.t_kv_heads, wl.t_head_dim, wl.prefix, T)


def test_hints_for_a_stable_cache_and_the_next_layer_change_nothing_but_time():
    """MASW_KV_STABLE (first tile requested ahead of the wait) and the next layer's L2 hint are scheduling hints: with
    them a chain of layer launches gives what each launch gives alone (deterministic schedule: bit for bit), and
    matches the oracle."""
    rng = inputs.rng_for(5, 0, 17)
    B, Hq, Hkv, D, P, T, L = 1, 32, 8, 128, 8192, 5, 3
    ks = [inputs.normal_bf16(rng, (B, Hkv, P + T, D)) for _ in range(L)]
    vs = [inputs.normal_bf16(rng, (B, Hkv, P + T, D)) for _ in range(L)]
    qs = [inputs.normal_bf16(rng, (B, T, Hq, D)) for _ in range(L)]
    K, V, Q = [dev_bf16(x) for x in ks], [dev_bf16(x) for x in vs], [dev_bf16(x) for x in qs]
    kv_len = torch.tensor([P + T], dtype=torch.int32, device="cuda")
    ws = binding.verify_workspace(K[0], kv_len, Hq, T)
    alone = [binding.verify_attend(K[l], V[l], kv_len, Q[l], workspace=ws, deterministic=True) for l in range(L)]
    alone = [(o.clone(), l.clone()) for o, l in alone]
    torch.cuda.synchronize()
    chained = [binding.verify_attend(K[l], V[l], kv_len, Q[l], workspace=ws, deterministic=True, stable_cache=True,
                                     next_kv=(K[l + 1], V[l + 1]) if l + 1 < L else None) for l in range(L)]
    for l in range(L):
        assert torch.equal(chained[l][0], alone[l][0]) and torch.equal(chained[l][1], alone[l][1])
        oref, lref = oracle.verify_attend(f64(qs[l]), f64(ks[l]), f64(vs[l]), [P + T])
        assert_attention_close(chained[l][0].cpu().numpy(), oref, chained[l][1].cpu().numpy(), lref, tag=f"hinted chain, layer {l}")


def test_sweep_batches():
    rng = inputs.rng_for(5, 0, 16)
    _case(rng, 4, 32, 8, 128, 4096, 2)
    _case(rng, 16, 32, 8, 128, 4096, 8)


def _paged_case(rng, B, Hq, Hkv, lens, T, extra_pages=3):
    """The same cache contiguous and scattered into a page pool in random order: identical attention."""
    D = 128
    cap = (max(lens) + 127) // 128 * 128
    kb, vb = inputs.normal_bf16(rng, (B, Hkv, cap, D)), inputs.normal_bf16(rng, (B, Hkv, cap, D))
    qb = inputs.normal_bf16(rng, (B, T, Hq, D))
    max_pages = cap // 128
    n_pages = B * max_pages + extra_pages
    perm = rng.permutation(n_pages)
    table = np.full((B, max_pages), -1, dtype=np.int32)
    kp = inputs.normal_bf16(rng, (n_pages, Hkv, 128, D))     # unused pages hold unrelated data
    vp = inputs.normal_bf16(rng, (n_pages, Hkv, 128, D))
    for b in range(B):
        for i in range((lens[b] + 127) // 128):
            pg = int(perm[b * max_pages + i])
            table[b, i] = pg
            kp[pg] = kb[b, :, 128 * i:128 * i + 128]
            vp[pg] = vb[b, :, 128 * i:128 * i + 128]
    kv_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
    og, lg, _ = binding.verify_attend_paged(dev_bf16(kp), dev_bf16(vp), torch.from_numpy(table).cuda(), kv_len, dev_bf16(qb))
    oref, lref = oracle.verify_attend(f64(qb), f64(kb), f64(vb), lens)
    assert_attention_close(og.cpu().numpy(), oref, lg.cpu().numpy(), lref, tag=f"paged verify B{B} lens{lens} T{T}")
    # and the contiguous entry point gives the same within the parity tolerance
    oc, _ = binding.verify_attend(dev_bf16(kb), dev_bf16(vb), kv_len, dev_bf16(qb))
    assert float((oc - og).abs().max()) <= 2e-2


def test_paged_cache_matches_the_oracle_and_the_contiguous_cache():
    """Page pool in random order, ragged lengths (the last page partly filled, sequences of different length),
    unused table entries -1, more pool pages than any sequence uses."""
    rng = inputs.rng_for(4, 0, 60)
    _paged_case(rng, 1, 8, 2, [1000], 5)
    _paged_case(rng, 3, 8, 2, [700, 129, 2048], 4)
    _paged_case(rng, 2, 16, 2, [8, 3000], 6)
    _paged_case(rng, 1, 32, 8, [6000], 5)
