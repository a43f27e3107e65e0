"""GPU parity: the verifier's attention over the FP8 (e4m3) paged cache against the CPU oracle.  The oracle is fed
the dequantised values exactly as the library defines them (fp16(e4m3 x fp16(scale)), q rounded to fp16), so the
attention tolerance of the bf16 path applies to the arithmetic alone."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_30252_b200 import binding, inputs
from helpers import assert_attention_close, dev_bf16, f64

pytestmark = pytest.mark.gpu


def _case(rng, B, Hq, Hkv, lens, T, extra_pages=2, q_scale=1.0, rel_tol=2e-3):
    D = 128
    cap = (max(lens) + 127) // 128 * 128
    max_pages = cap // 128
    n_pages = B * max_pages + extra_pages
    pool_k = rng.standard_normal((n_pages, Hkv, 128, D)).astype(np.float32)
    pool_v = rng.standard_normal((n_pages, Hkv, 128, D)).astype(np.float32)
    pool_v *= rng.uniform(0.2, 3.0, size=(n_pages, Hkv, 1, 1)).astype(np.float32)      # pages with different scales
    kb, ks = inputs.quantize_e4m3_pages(pool_k)
    vb, vs = inputs.quantize_e4m3_pages(pool_v)
    perm = rng.permutation(n_pages)
    table = np.full((B, max_pages), -1, dtype=np.int32)
    for b in range(B):
        for i in range((lens[b] + 127) // 128):
            table[b, i] = int(perm[b * max_pages + i])
    qb = inputs.normal_bf16(rng, (B, T, Hq, D), std=q_scale)
    # the oracle's inputs: dequantised pages gathered into contiguous caches, q rounded to fp16
    kd = oracle.dequantize_e4m3(kb, ks[:, :, None, None])
    vd = oracle.dequantize_e4m3(vb, vs[:, :, None, None])
    K = np.zeros((B, Hkv, cap, D)); V = np.zeros((B, Hkv, cap, D))
    for b in range(B):
        for i in range((lens[b] + 127) // 128):
            K[b, :, 128 * i:128 * i + 128] = kd[table[b, i]]
            V[b, :, 128 * i:128 * i + 128] = vd[table[b, i]]
    oref, lref = oracle.verify_attend(oracle.fp16_round(f64(qb)), K, V, lens)
    kv_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    args = (torch.from_numpy(kb).cuda(), torch.from_numpy(vb).cuda(), torch.from_numpy(ks).cuda(), torch.from_numpy(vs).cuda(),
            torch.from_numpy(table).cuda(), kv_len, dev_bf16(qb))
    og, lg, ws = binding.verify_attend_fp8(*args, status=status)
    assert int(status.item()) == 0
    res = assert_attention_close(og.cpu().numpy(), oref, lg.cpu().numpy(), lref, tag=f"fp8 verify B{B} lens{lens} T{T}", rel_tol=rel_tol)
    # the scratch is reusable, and the deterministic schedule repeats bit for bit
    od, ld, _ = binding.verify_attend_fp8(*args, workspace=ws, deterministic=True)
    od2, ld2, _ = binding.verify_attend_fp8(*args, workspace=ws, deterministic=True)
    assert torch.equal(od, od2) and torch.equal(ld, ld2)
    assert_attention_close(od.cpu().numpy(), oref, ld.cpu().numpy(), lref, tag="fp8 verify, deterministic", rel_tol=rel_tol)
    return res


def test_small_caches_ragged_lengths_and_random_page_order():
    rng = inputs.rng_for(4, 0, 80)
    _case(rng, 1, 8, 2, [1000], 5)
    _case(rng, 3, 8, 2, [700, 129, 2048], 4)
    _case(rng, 2, 16, 2, [8, 3000], 2)
    _case(rng, 1, 32, 8, [6000], 5)


def test_probabilities_in_fp16_leave_a_wide_margin():
    """fp16 probabilities carry 11 significant bits (the bf16 cache's kernel: 8), so the arithmetic error is far
    below the 2e-3 tolerance."""
    rng = inputs.rng_for(4, 0, 81)
    _, rel = _case(rng, 1, 8, 2, [4096], 5)
    assert rel < 5e-4, rel
    _case(rng, 1, 8, 2, [4096], 5, q_scale=6.0)          # peaky scores


@pytest.mark.parametrize("B", [1, 4])
def test_full_size_32k_layer(B):
    """The 8B-shaped target at 32K (the benchmark's FP8 comparison point), all heads and rows of one layer."""
    rng = inputs.rng_for(3, 0, 82 + B)
    _case(rng, B, 32, 8, [32768 + 5] * B, 5, extra_pages=1)


def test_arguments_are_validated_before_launch():
    kp = torch.zeros((4, 2, 128, 128), dtype=torch.uint8, device="cuda")
    sc = torch.ones((4, 2), dtype=torch.float32, device="cuda")
    table = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    kv_len = torch.tensor([300], dtype=torch.int32, device="cuda")
    q = torch.zeros((1, 9, 8, 128), dtype=torch.bfloat16, device="cuda")      # 9 rows x group 4 > 32
    with pytest.raises(binding.MaswError) as ei:
        binding.verify_attend_fp8(kp, kp, sc, sc, table, kv_len, q)
    assert ei.value.code == binding.MASW_EINVAL
