"""The allocation-free accept/reject entry point (collected last on purpose: if it fails, a run that
stops at the first failure has already run every other test).

accept_reject_static serves callers that cannot allocate device memory where the accept/reject
decision is taken (all memory already handed to their own pool, or cudaMalloc ruled out because it
would stall the device in the middle of decoding).  Its scratch is a fixed array inside the library,
shared by every call on the device, so the test runs two calls back to back on different inputs and
compares each with the workspace-taking entry point and with the CPU oracle's decisions: the second
call must not be disturbed by what the first one left behind."""
import numpy as np
import pytest
import torch

import oracle
from paper_2608_30252_b200 import binding, inputs
from helpers import dev_bf16, host_bits

pytestmark = pytest.mark.gpu


def _inputs(rng, B, gamma, V):
    tl, dl = inputs.logits_pair(rng, B, gamma, V, target_std=2.0, noise_std=0.7)
    z = np.exp(inputs.bf16_bits_to_f32(dl).astype(np.float64))
    q = z / z.sum(-1, keepdims=True)
    toks = np.stack([[rng.choice(V, p=q[b, i]) for i in range(gamma)] for b in range(B)]).astype(np.int32)
    u = inputs.uniforms_24bit(rng, (B, gamma + 1))
    return dev_bf16(tl), dev_bf16(dl), torch.from_numpy(toks).cuda(), torch.from_numpy(u).cuda()


@pytest.mark.parametrize("temperature", [0.0, 1.0])
def test_two_calls_in_a_row_match_the_workspace_entry_point(temperature):
    rng = inputs.rng_for(1, 0, 30)
    cases = [_inputs(rng, 3, 5, 4000), _inputs(rng, 2, 4, 32000)]      # different shapes share the one scratch array
    expected = [binding.accept_reject(tl, dl, toks, u, temperature) for tl, dl, toks, u in cases]
    torch.cuda.synchronize()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = [binding.accept_reject_static(tl, dl, toks, u, temperature, status=status) for tl, dl, toks, u in cases]
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for (n_ref, out_ref), (n, out) in zip(expected, got):
        assert torch.equal(n, n_ref) and torch.equal(out, out_ref)      # integer decisions: bit-exact
    # and directly against the oracle's decisions on the same logits, tokens and uniforms
    for (tl, dl, toks, u), (n, out) in zip(cases, got):
        f = lambda t: oracle.bf16_bits_to_f64(host_bits(t))
        n_ref, out_ref = oracle.accept_reject(f(tl), f(dl), toks.cpu().numpy(), u.cpu().numpy(), temperature)
        assert np.array_equal(n.cpu().numpy(), n_ref) and np.array_equal(out.cpu().numpy(), out_ref)
    # and once more in the opposite order, so each shape also follows the other one
    again = [binding.accept_reject_static(tl, dl, toks, u, temperature) for tl, dl, toks, u in reversed(cases)]
    for (n_ref, out_ref), (n, out) in zip(reversed(expected), again):
        assert torch.equal(n, n_ref) and torch.equal(out, out_ref)


def test_sizes_beyond_the_built_in_scratch_are_rejected():
    tl = torch.zeros((65, 3, 16), dtype=torch.bfloat16, device="cuda")
    toks = torch.zeros((65, 2), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.MaswError) as ei:
        binding.accept_reject_static(tl, None, toks, None, 0.0)
    assert ei.value.code == binding.MASW_ECAPACITY and "batch" in str(ei.value)
    tl = torch.zeros((1, 18, 16), dtype=torch.bfloat16, device="cuda")
    toks = torch.zeros((1, 17), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.MaswError) as ei:
        binding.accept_reject_static(tl, None, toks, None, 0.0)
    assert ei.value.code == binding.MASW_ECAPACITY
